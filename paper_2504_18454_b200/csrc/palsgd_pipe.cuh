// Persistent, warp-specialised form of the fused inner step.
//
// One CTA per SM loops over its work items.  A producer warp streams each
// item's inputs (g, x, m, v -- or x, x_g for a pull) from HBM into a ring of
// shared-memory stages with 1-D bulk asynchronous copies (the TMA engine,
// cp.async.bulk + mbarrier transaction counts; no multicast, this GPU's own
// memory only), several items ahead of the consumer warps, which read a stage
// into registers, release it, do the arithmetic and write the results back
// with 128-bit streaming stores.  The copies in flight are bounded by shared
// memory, not by registers or occupancy, and there is one prologue and one
// counter tick per CTA instead of one per item.
//
// Only full, 16-byte-aligned chunks (the first n_full entries of the chunk
// table) go through the ring; the ragged rest is handled by the same CTAs with
// the register path once the ring has drained.
//
// Every wait on an mbarrier is bounded: on expiry the thread records an error
// in the device state and leaves its loop, so a fault can never hang the GPU.
#pragma once
#include "palsgd_kernels.cuh"

namespace palsgd {

constexpr uint32_t kPipeMaxStages = 8;
constexpr uint32_t kPipeSpinLimit = 1u << 22;      // polls before a wait gives up (order of a second)
constexpr uint32_t kErrPipeFullTimeout  = 1;       // DevState::error codes
constexpr uint32_t kErrPipeEmptyTimeout = 2;

struct PipeDesc {                 // what the consumers need to know about the item in a stage
    float*          x;
    float*          m;
    float*          v;
    __nv_bfloat16*  w;
    uint32_t        k;
    uint32_t        pull;
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false when the phase did not complete within the poll limit.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity)
{
    for (uint32_t i = 0; i < kPipeSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 1024) __nanosleep(128);
    }
    return false;
}
// global -> shared bulk copy of `bytes` (multiple of 16, both sides 16-byte aligned),
// completion counted on `bar`
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst_smem)), "l"(__cvta_generic_to_global(src_gmem)), "r"(bytes),
                   "r"(smem_addr(bar)) : "memory");
}

// NC consumer threads + one producer warp.  Stage layout (T = kChunkElems):
//   gradient step: x @0, m @4T, [v @8T,] g behind them;   pull: x @0, x_g @4T.
template <int INNER, int PREC, int NC>
__global__ void __launch_bounds__(NC + 32, 1)
palsgd_inner_pipe_kernel(const __grid_constant__ InnerArgs a, uint32_t n_stages, uint32_t stage_bytes)
{
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ __align__(8) uint64_t full_bar[kPipeMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kPipeMaxStages];
    __shared__ PipeDesc desc[kPipeMaxStages];
    __shared__ unsigned char s_pull[kMaxWorkers];
    __shared__ float s_bc1[kMaxWorkers], s_bc2[kMaxWorkers];

    constexpr uint32_t T = kStageElems;
    constexpr uint32_t UN = T / 4 / NC;                  // 4-element units per consumer thread and stage
    static_assert(UN >= 1 && UN * 4 * NC == T, "consumer count must divide the chunk");
    constexpr uint32_t kGradOff = (INNER == 0 ? 12u : 8u) * T;     // byte offset of g in a stage
    constexpr uint32_t kGradBytes = (PREC ? 2u : 4u) * T;

    const Tables& tb = a.tb;
    const uint32_t K = tb.K;
    DevState* st = tb.st;
    const unsigned long long t = st->t;
    const uint32_t tid = threadIdx.x;

    if (tid < K) {
        const bool pull = draw_pull(a.seed, t, tid, a.thr);
        s_pull[tid] = pull;
        if (INNER == 0 && !pull) {
            s_bc1[tid] = (float)(1.0 - st->pow1[tid] * a.beta1);
            s_bc2[tid] = (float)(1.0 - st->pow2[tid] * a.beta2);
        }
    }
    if (tid == 0) {
        for (uint32_t s = 0; s < n_stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], NC / 32); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const uint32_t R = tb.chunk_elems / T;               // stage-sized pieces per full chunk
    const uint64_t n_items = (uint64_t)tb.n_full * K * R;

    if (tid < 32) {
        // ------------------------------------------------ producer (one elected lane)
        if (tid == 0) {
            uint32_t s = 0, round = 0;
            for (uint64_t item = blockIdx.x; item < n_items; item += gridDim.x) {
                if (round > 0 && !mbar_wait(&empty_bar[s], (round - 1) & 1u)) {
                    atomicExch(&st->error, kErrPipeEmptyTimeout);
                    break;
                }
                const uint32_t k = (uint32_t)(item % K);
                Chunk ch = tb.chunks[item / K / R];
                ch.off += (uint64_t)((item / K) % R) * T;
                const uint32_t seg = ch.seg & ~kSegVecFlag;
                const size_t pi = (size_t)k * tb.n_seg + seg;
                float* x = tb.xf[pi] + ch.off;
                const bool pull = s_pull[k];
                PipeDesc d;
                d.x = x; d.k = k; d.pull = pull;
                d.m = tb.m[pi] + ch.off;
                d.v = INNER == 0 ? tb.v[pi] + ch.off : nullptr;
                d.w = PREC ? tb.xw[pi] + ch.off : nullptr;
                desc[s] = d;
                unsigned char* sb = ring + (size_t)s * stage_bytes;
                if (pull) {
                    mbar_arrive_expect_tx(&full_bar[s], 8u * T);
                    bulk_load(sb, x, 4u * T, &full_bar[s]);
                    bulk_load(sb + 4u * T, tb.global[seg] + ch.off, 4u * T, &full_bar[s]);
                } else {
                    const char* g = static_cast<const char*>(tb.grad[pi]) + ch.off * (PREC ? 2u : 4u);
                    mbar_arrive_expect_tx(&full_bar[s], kGradOff + kGradBytes);
                    bulk_load(sb, x, 4u * T, &full_bar[s]);
                    bulk_load(sb + 4u * T, d.m, 4u * T, &full_bar[s]);
                    if (INNER == 0) bulk_load(sb + 8u * T, d.v, 4u * T, &full_bar[s]);
                    bulk_load(sb + kGradOff, g, kGradBytes, &full_bar[s]);
                }
                if (++s == n_stages) { s = 0; ++round; }
            }
        }
    } else {
        // ------------------------------------------------ consumers
        const uint32_t ct = tid - 32;
        uint32_t s = 0, phase = 0;
        for (uint64_t item = blockIdx.x; item < n_items; item += gridDim.x) {
            if (!mbar_wait(&full_bar[s], phase)) {
                atomicExch(&st->error, kErrPipeFullTimeout);
                break;
            }
            const PipeDesc d = desc[s];
            const unsigned char* sb = ring + (size_t)s * stage_bytes;
            const float4* sx = reinterpret_cast<const float4*>(sb);
            if (d.pull) {
                const float4* sq = reinterpret_cast<const float4*>(sb + 4u * T);
                float4 X[UN], Q[UN];
#pragma unroll
                for (uint32_t h = 0; h < UN; ++h) { X[h] = sx[ct + NC * h]; Q[h] = sq[ct + NC * h]; }
                __syncwarp();
                if ((ct & 31u) == 0) mbar_arrive(&empty_bar[s]);
#pragma unroll
                for (uint32_t h = 0; h < UN; ++h) {
                    const uint32_t j = ct + NC * h;
                    PALSGD_FOR4(comp(X[h], c) = pull_elem(compv(X[h], c), compv(Q[h], c), a.beta_pull))
                    st_stream(reinterpret_cast<float4*>(d.x) + j, X[h]);
                    if (PREC) st_stream(reinterpret_cast<uint2*>(d.w) + j,
                                        make_uint2(pack_bf16x2(X[h].x, X[h].y), pack_bf16x2(X[h].z, X[h].w)));
                }
            } else {
                const float4* sm = reinterpret_cast<const float4*>(sb + 4u * T);
                const float4* sv = reinterpret_cast<const float4*>(sb + 8u * T);
                float4 X[UN], M[UN], V[UN];
                float G[UN][4];
#pragma unroll
                for (uint32_t h = 0; h < UN; ++h) {
                    const uint32_t j = ct + NC * h;
                    X[h] = sx[j]; M[h] = sm[j];
                    if (INNER == 0) V[h] = sv[j];
                    if (PREC) {
                        const uint2 gh = reinterpret_cast<const uint2*>(sb + kGradOff)[j];
                        G[h][0] = bf16_bits_to_f32(gh.x & 0xFFFFu); G[h][1] = __uint_as_float(gh.x & 0xFFFF0000u);
                        G[h][2] = bf16_bits_to_f32(gh.y & 0xFFFFu); G[h][3] = __uint_as_float(gh.y & 0xFFFF0000u);
                    } else {
                        const float4 gf = reinterpret_cast<const float4*>(sb + kGradOff)[j];
                        G[h][0] = gf.x; G[h][1] = gf.y; G[h][2] = gf.z; G[h][3] = gf.w;
                    }
                }
                __syncwarp();
                if ((ct & 31u) == 0) mbar_arrive(&empty_bar[s]);
                const AdamScalars as{a.b1, a.b2, a.omb1, a.omb2, s_bc1[d.k], s_bc2[d.k], a.decay, a.lr, a.eps};
                const SgdScalars  ss{a.mu, a.wd, a.lr};
#pragma unroll
                for (uint32_t h = 0; h < UN; ++h) {
                    const uint32_t j = ct + NC * h;
                    if (INNER == 0) {
                        PALSGD_FOR4(adamw_elem(G[h][c], comp(X[h], c), comp(M[h], c), comp(V[h], c), as))
                        st_stream(reinterpret_cast<float4*>(d.v) + j, V[h]);
                    } else {
                        PALSGD_FOR4(sgdm_elem(G[h][c], comp(X[h], c), comp(M[h], c), ss))
                    }
                    st_stream(reinterpret_cast<float4*>(d.x) + j, X[h]);
                    st_stream(reinterpret_cast<float4*>(d.m) + j, M[h]);
                    if (PREC) st_stream(reinterpret_cast<uint2*>(d.w) + j,
                                        make_uint2(pack_bf16x2(X[h].x, X[h].y), pack_bf16x2(X[h].z, X[h].w)));
                }
            }
            if (++s == n_stages) { s = 0; phase ^= 1u; }
        }

        // ---- the ragged rest (partial chunks, unaligned segments): register path
        const uint64_t n_rest = (uint64_t)(tb.n_chunks - tb.n_full) * K;
        for (uint64_t r = blockIdx.x; r < n_rest; r += gridDim.x) {
            const uint32_t k = (uint32_t)(r % K);
            const Chunk ch = tb.chunks[tb.n_full + r / K];
            if (s_pull[k]) {
                pull_item<PREC, 1, NC>(ct, tb, k, ch, a.beta_pull);
            } else {
                const AdamScalars as{a.b1, a.b2, a.omb1, a.omb2, s_bc1[k], s_bc2[k], a.decay, a.lr, a.eps};
                const SgdScalars  ss{a.mu, a.wd, a.lr};
                grad_item<INNER, PREC, 1, NC>(ct, tb, k, ch, as, ss);
            }
        }
    }

    // ---- counter tick by the last CTA
    __syncthreads();
    if (tid == 0) {
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
            __threadfence();
        }
    }
}


// ---------------------------------------------------------------------------
// Second form: ALL warps of the CTA consume (one 4-element unit per thread and
// stage), and thread 0 also plays producer at the top of each iteration: it
// refills the stage the CTA drained one iteration ago, with the item
// n_stages - 1 ahead, whose table entries it fetched an iteration earlier.
// More resident warps hide the latency of the division / square-root chains.
struct PipeMeta {                 // producer-side view of one item (pointers already offset)
    float* x; float* m; float* v; __nv_bfloat16* w; const char* g; const float* xg;
    uint32_t k; uint32_t valid;
};

template <int INNER, int PREC>
__device__ __forceinline__ PipeMeta pipe_fetch_meta(const Tables& tb, uint64_t item, uint64_t n_items)
{
    PipeMeta mt;
    mt.valid = item < n_items;
    if (!mt.valid) { mt.x = mt.m = mt.v = nullptr; mt.w = nullptr; mt.g = nullptr; mt.xg = nullptr; mt.k = 0; return mt; }
    const uint32_t K = tb.K;
    const uint32_t R = tb.chunk_elems / kStageElems;
    mt.k = (uint32_t)(item % K);
    Chunk ch = tb.chunks[item / K / R];
    ch.off += (uint64_t)((item / K) % R) * kStageElems;
    const uint32_t seg = ch.seg & ~kSegVecFlag;
    const size_t pi = (size_t)mt.k * tb.n_seg + seg;
    mt.x = tb.xf[pi] + ch.off;
    mt.m = tb.m[pi] + ch.off;
    mt.v = INNER == 0 ? tb.v[pi] + ch.off : nullptr;
    mt.w = PREC ? tb.xw[pi] + ch.off : nullptr;
    mt.g = static_cast<const char*>(tb.grad[pi]) + ch.off * (PREC ? 2u : 4u);
    mt.xg = tb.global[seg] + ch.off;
    return mt;
}

template <int INNER, int PREC>
__global__ void __launch_bounds__(1024, 1)
palsgd_inner_pipe_all_kernel(const __grid_constant__ InnerArgs a, uint32_t n_stages, uint32_t stage_bytes)
{
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ __align__(8) uint64_t full_bar[kPipeMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kPipeMaxStages];
    __shared__ PipeDesc desc[kPipeMaxStages];
    __shared__ unsigned char s_pull[kMaxWorkers];
    __shared__ float s_bc1[kMaxWorkers], s_bc2[kMaxWorkers];

    constexpr uint32_t T = kStageElems;
    constexpr uint32_t NC = 1024;
    static_assert(T == 4 * NC, "one 4-element unit per thread and stage");
    constexpr uint32_t kGradOff = (INNER == 0 ? 12u : 8u) * T;
    constexpr uint32_t kGradBytes = (PREC ? 2u : 4u) * T;

    const Tables& tb = a.tb;
    const uint32_t K = tb.K;
    DevState* st = tb.st;
    const unsigned long long t = st->t;
    const uint32_t tid = threadIdx.x;

    if (tid < K) {
        const bool pull = draw_pull(a.seed, t, tid, a.thr);
        s_pull[tid] = pull;
        if (INNER == 0 && !pull) {
            s_bc1[tid] = (float)(1.0 - st->pow1[tid] * a.beta1);
            s_bc2[tid] = (float)(1.0 - st->pow2[tid] * a.beta2);
        }
    }
    if (tid == 0) {
        for (uint32_t s = 0; s < n_stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], NC / 32); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const uint64_t n_items = (uint64_t)tb.n_full * K * (tb.chunk_elems / T);
    const uint64_t G = gridDim.x;

    // issue the copies of one item into stage s (thread 0 only)
    auto issue = [&](const PipeMeta& mt, uint32_t s) {
        const bool pull = s_pull[mt.k];
        PipeDesc d;
        d.x = mt.x; d.m = mt.m; d.v = mt.v; d.w = mt.w; d.k = mt.k; d.pull = pull;
        desc[s] = d;
        unsigned char* sb = ring + (size_t)s * stage_bytes;
        if (pull) {
            mbar_arrive_expect_tx(&full_bar[s], 8u * T);
            bulk_load(sb, mt.x, 4u * T, &full_bar[s]);
            bulk_load(sb + 4u * T, mt.xg, 4u * T, &full_bar[s]);
        } else {
            mbar_arrive_expect_tx(&full_bar[s], kGradOff + kGradBytes);
            bulk_load(sb, mt.x, 4u * T, &full_bar[s]);
            bulk_load(sb + 4u * T, mt.m, 4u * T, &full_bar[s]);
            if (INNER == 0) bulk_load(sb + 8u * T, mt.v, 4u * T, &full_bar[s]);
            bulk_load(sb + kGradOff, mt.g, kGradBytes, &full_bar[s]);
        }
    };

    // prologue: fill n_stages - 1 stages, fetch the table entries of the next item
    PipeMeta next;
    next.valid = 0;
    if (tid == 0) {
        for (uint32_t j = 0; j + 1 < n_stages; ++j) {
            const PipeMeta mt = pipe_fetch_meta<INNER, PREC>(tb, blockIdx.x + j * G, n_items);
            if (mt.valid) issue(mt, j);
        }
        next = pipe_fetch_meta<INNER, PREC>(tb, blockIdx.x + (uint64_t)(n_stages - 1) * G, n_items);
    }

    // Item number `it` of this CTA lives in stage it % n_stages.  At iteration `it` thread 0 issues
    // item it + n_stages - 1 into the stage that item it - 1 occupied, once every warp has released it.
    uint32_t s = 0, phase = 0;                  // stage and parity of the item being consumed
    uint32_t rs = 0, rphase = 0;                // stage of item it - 1 and the parity of its release
    bool failed = false;
    uint64_t it = 0;
    for (uint64_t item = blockIdx.x; item < n_items; item += G, ++it) {
        if (tid == 0 && next.valid) {
            const bool ok = it == 0 ? true : mbar_wait(&empty_bar[rs], rphase);
            if (ok) {
                issue(next, it == 0 ? n_stages - 1 : rs);
                next = pipe_fetch_meta<INNER, PREC>(tb, item + (uint64_t)n_stages * G, n_items);
            } else {
                atomicExch(&st->error, kErrPipeEmptyTimeout);
                next.valid = 0;
            }
        }
        if (it > 0 && ++rs == n_stages) { rs = 0; rphase ^= 1u; }
        __syncwarp();
        if (!mbar_wait(&full_bar[s], phase)) { atomicExch(&st->error, kErrPipeFullTimeout); failed = true; break; }
        const PipeDesc d = desc[s];
        const unsigned char* sb = ring + (size_t)s * stage_bytes;
        float4 X = reinterpret_cast<const float4*>(sb)[tid];
        if (d.pull) {
            const float4 Q = reinterpret_cast<const float4*>(sb + 4u * T)[tid];
            __syncwarp();
            if ((tid & 31u) == 0) mbar_arrive(&empty_bar[s]);
            PALSGD_FOR4(comp(X, c) = pull_elem(compv(X, c), compv(Q, c), a.beta_pull))
            st_stream(reinterpret_cast<float4*>(d.x) + tid, X);
        } else {
            float4 M = reinterpret_cast<const float4*>(sb + 4u * T)[tid];
            float4 V;
            if (INNER == 0) V = reinterpret_cast<const float4*>(sb + 8u * T)[tid];
            float G4[4];
            if (PREC) {
                const uint2 gh = reinterpret_cast<const uint2*>(sb + kGradOff)[tid];
                G4[0] = bf16_bits_to_f32(gh.x & 0xFFFFu); G4[1] = __uint_as_float(gh.x & 0xFFFF0000u);
                G4[2] = bf16_bits_to_f32(gh.y & 0xFFFFu); G4[3] = __uint_as_float(gh.y & 0xFFFF0000u);
            } else {
                const float4 gf = reinterpret_cast<const float4*>(sb + kGradOff)[tid];
                G4[0] = gf.x; G4[1] = gf.y; G4[2] = gf.z; G4[3] = gf.w;
            }
            __syncwarp();
            if ((tid & 31u) == 0) mbar_arrive(&empty_bar[s]);
            if (INNER == 0) {
                const AdamScalars as{a.b1, a.b2, a.omb1, a.omb2, s_bc1[d.k], s_bc2[d.k], a.decay, a.lr, a.eps};
                PALSGD_FOR4(adamw_elem(G4[c], comp(X, c), comp(M, c), comp(V, c), as))
                st_stream(reinterpret_cast<float4*>(d.v) + tid, V);
            } else {
                const SgdScalars ss{a.mu, a.wd, a.lr};
                PALSGD_FOR4(sgdm_elem(G4[c], comp(X, c), comp(M, c), ss))
            }
            st_stream(reinterpret_cast<float4*>(d.x) + tid, X);
            st_stream(reinterpret_cast<float4*>(d.m) + tid, M);
        }
        if (PREC) st_stream(reinterpret_cast<uint2*>(d.w) + tid,
                            make_uint2(pack_bf16x2(X.x, X.y), pack_bf16x2(X.z, X.w)));
        if (++s == n_stages) { s = 0; phase ^= 1u; }
    }

    // ---- the ragged rest: register path
    if (!failed) {
        const uint64_t n_rest = (uint64_t)(tb.n_chunks - tb.n_full) * K;
        for (uint64_t r = blockIdx.x; r < n_rest; r += G) {
            const uint32_t k = (uint32_t)(r % K);
            const Chunk ch = tb.chunks[tb.n_full + r / K];
            if (s_pull[k]) {
                pull_item<PREC, 1, NC>(tid, tb, k, ch, a.beta_pull);
            } else {
                const AdamScalars as{a.b1, a.b2, a.omb1, a.omb2, s_bc1[k], s_bc2[k], a.decay, a.lr, a.eps};
                const SgdScalars  ss{a.mu, a.wd, a.lr};
                grad_item<INNER, PREC, 1, NC>(tid, tb, k, ch, as, ss);
            }
        }
    }

    __syncthreads();
    if (tid == 0) {
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
            __threadfence();
        }
    }
}

}  // namespace palsgd
