// Host controller and C ABI of the PALSGD library (see include/palsgd.h).
//
// The controller validates arguments, fuses adjacent tensors into segments,
// builds the chunk table and pointer tables once, forms the per-call scalars
// in binary64, and launches one kernel per call.  Counters that the kernels
// need (t, s_k, beta^s_k) live on the device; the host keeps a mirror of t and
// n_outer for the "(t+1) mod H" test.
#include "../../include/palsgd.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "palsgd_kernels.cuh"
#include "palsgd_norm.cuh"
#include "palsgd_pipe.cuh"

using namespace palsgd;

struct Segment {
    size_t   first_tensor;
    size_t   n_tensors;
    uint64_t numel;
};

struct palsgd_ctx {
    palsgd_config cfg{};
    size_t n_tensors = 0;
    std::vector<uint64_t> numel;
    std::vector<Segment> segs;
    // host copies of the caller's pointer arrays (for the host-buffer entry point)
    std::vector<const void*> h_grad_dev;     // [K*n_tensors] device gradient pointers
    std::vector<float*> h_global_dev;        // [n_tensors]
    // device tables
    void* d_blob = nullptr;                  // one allocation holding everything below
    Tables tb{};
    uint64_t P = 0;
    // host mirrors
    uint64_t t = 0, n_outer = 0, launches = 0;
    uint64_t thr = 0;
    int grid_cap_inner = 0, grid_cap_outer = 0;   // 0 = one CTA per work item
    int inner_variant = 0;                        // launch shape of the inner kernel, 0 = default
    int pipe_stages = 0;                          // ring depth of the pipelined kernel, 0 = as many as fit
    int chunk_major = 0;                          // work-item order of the register-path inner kernel
    uint32_t chunk_elems = kChunkElems;           // elements per chunk-table entry (fixed at init)
    uint32_t outer_sub_elems = kOuterSubElems;    // elements per work item of the outer kernel
    uint32_t ddp_sub_elems = kDdpSubElems;        // elements per work item of the DDP warm-up kernel
    int ddp_variant = 0;                          // 0 = default, 1 = per-thread stores, 2 = staged bulk stores
    int outer_variant = 0;                        // the same for the outer kernel
    int outer_dynamic = -1;                       // outer / DDP kernels: CTAs per SM of a persistent grid, 0 = one CTA
                                                  // per item, -1 = default (outer: 0, DDP: 4; measured)
    double max_grad_norm = 0.0;                   // global-norm clip threshold, 0 = off
    double outer_lr = 0.0;                        // OuterOPT learning rate of the next sync
    double opow1 = 1.0, opow2 = 1.0;              // outer_beta^n_outer (AdamW as OuterOPT), running products
    cudaStream_t copy_stream = nullptr;           // palsgd_step_host: host -> device copies run here ...
    std::vector<cudaEvent_t> copy_done;           // ... and signal worker k's gradient with copy_done[k]
    cudaEvent_t copy_may_start = nullptr;         // recorded on the caller's stream before the copies begin
    cudaGraphExec_t cycle_exec = nullptr;         // captured H-step cycle (palsgd_cycle_capture) or nullptr
    uint64_t cycle_launches = 0;                  // kernels inside one captured cycle
    int sm_count = 0, smem_optin = 0;             // device attributes read at init
    std::string cuda_err;
};

namespace {

thread_local std::string g_noctx_err;

int cuda_fail(palsgd_ctx* ctx, cudaError_t e, const char* what)
{
    std::string msg = std::string(what) + ": " + cudaGetErrorString(e);
    if (ctx) ctx->cuda_err = msg; else g_noctx_err = msg;
    return PALSGD_ECUDA;
}

#define PALSGD_CUDA(ctx, call)                                            \
    do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return cuda_fail((ctx), e_, #call); } while (0)

inline bool finite_nonneg(double v) { return std::isfinite(v) && v >= 0.0; }
inline size_t elem_size_param(int prec) { return prec == PALSGD_PREC_BF16_MASTER ? 2 : 4; }
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

uint64_t threshold_of(double p) { return (uint64_t)std::floor(p * 4294967296.0); }

int validate_config(const palsgd_config* c)
{
    if (!c) return PALSGD_EINVAL;
    if (c->K == 0 || c->K > PALSGD_MAX_WORKERS) return PALSGD_EINVAL;
    if (c->H == 0) return PALSGD_EINVAL;
    if (!(c->p >= 0.0 && c->p <= 1.0)) return PALSGD_EINVAL;
    if (c->inner != PALSGD_INNER_ADAMW && c->inner != PALSGD_INNER_SGDM) return PALSGD_EINVAL;
    if (c->precision != PALSGD_PREC_FP32 && c->precision != PALSGD_PREC_BF16_MASTER) return PALSGD_EINVAL;
    if (c->outer_nesterov != 0 && c->outer_nesterov != 1) return PALSGD_EINVAL;
    if (c->inner == PALSGD_INNER_ADAMW) {
        if (!(c->beta1 >= 0.0 && c->beta1 < 1.0) || !(c->beta2 >= 0.0 && c->beta2 < 1.0)) return PALSGD_EINVAL;
        if (!finite_nonneg(c->eps)) return PALSGD_EINVAL;
    } else {
        if (!finite_nonneg(c->momentum)) return PALSGD_EINVAL;
    }
    if (!finite_nonneg(c->weight_decay)) return PALSGD_EINVAL;
    if (!std::isfinite(c->outer_lr) || !finite_nonneg(c->outer_momentum)) return PALSGD_EINVAL;
    if (c->outer_opt != PALSGD_OUTER_SGD && c->outer_opt != PALSGD_OUTER_ADAMW) return PALSGD_EINVAL;
    if (c->outer_opt == PALSGD_OUTER_ADAMW) {
        if (!(c->outer_beta1 >= 0.0 && c->outer_beta1 < 1.0) || !(c->outer_beta2 >= 0.0 && c->outer_beta2 < 1.0))
            return PALSGD_EINVAL;
        if (!finite_nonneg(c->outer_eps) || !finite_nonneg(c->outer_weight_decay)) return PALSGD_EINVAL;
    }
    return PALSGD_OK;
}

// Pointer of buffer kind `kind` for (k, j); kinds: 0 param 1 grad 2 master 3 m 4 v
const void* buf_ptr(const palsgd_buffers* b, int kind, size_t idx)
{
    switch (kind) {
        case 0: return b->param[idx];
        case 1: return b->grad[idx];
        case 2: return b->master[idx];
        case 3: return b->m[idx];
        default: return b->v[idx];
    }
}

template <typename F>
int launch_checked(palsgd_ctx* ctx, F&& launch)
{
    launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "kernel launch");
    ctx->launches += 1;
    return PALSGD_OK;
}

unsigned grid_for(uint64_t n_items, int cap)
{
    uint64_t g = n_items;
    if (cap > 0 && g > (uint64_t)cap) g = (uint64_t)cap;
    if (g > 0x7FFFFFFFull) g = 0x7FFFFFFFull;
    return (unsigned)(g == 0 ? 1 : g);
}

OuterArgs outer_args(const palsgd_ctx* ctx)
{
    OuterArgs a{};
    a.tb = ctx->tb;
    a.mu = (float)ctx->cfg.outer_momentum;
    a.lr = (float)ctx->outer_lr;
    a.Kf = (float)ctx->cfg.K;
    a.nesterov = ctx->cfg.outer_nesterov;
    if (ctx->cfg.outer_opt == PALSGD_OUTER_ADAMW) {          // scalars of outer step n_outer + 1
        const palsgd_config& c = ctx->cfg;
        a.ob1 = (float)c.outer_beta1;
        a.ob2 = (float)c.outer_beta2;
        a.oomb1 = (float)(1.0 - c.outer_beta1);
        a.oomb2 = (float)(1.0 - c.outer_beta2);
        a.obc1 = (float)(1.0 - ctx->opow1 * c.outer_beta1);
        a.obc2 = (float)(1.0 - ctx->opow2 * c.outer_beta2);
        a.odecay = (float)(1.0 - ctx->outer_lr * c.outer_weight_decay);
        a.oeps = (float)c.outer_eps;
    }
    a.sub_elems = ctx->outer_sub_elems;
    a.parts = (ctx->chunk_elems + a.sub_elems - 1) / a.sub_elems;
    return a;
}

// Launch shapes of the fused inner kernel: U = 128-bit loads in flight per
// stream and thread, MINB = CTAs per SM the register budget is held to.
template <int INNER, int PREC>
void launch_inner_variant(int variant, unsigned grid, cudaStream_t s, const InnerArgs& a)
{
    switch (variant) {
        case 1:  palsgd_inner_kernel<INNER, PREC, 1, 4><<<grid, kThreads, 0, s>>>(a); break;
        case 2:  palsgd_inner_kernel<INNER, PREC, 1, 3><<<grid, kThreads, 0, s>>>(a); break;
        case 3:  palsgd_inner_kernel<INNER, PREC, 2, 2><<<grid, kThreads, 0, s>>>(a); break;
        case 4:  palsgd_inner_kernel<INNER, PREC, 2, 3><<<grid, kThreads, 0, s>>>(a); break;
        case 5:  palsgd_inner_kernel<INNER, PREC, 4, 1><<<grid, kThreads, 0, s>>>(a); break;
        case 6:  palsgd_inner_kernel<INNER, PREC, 1, 6><<<grid, kThreads, 0, s>>>(a); break;
        case 7:  palsgd_inner_kernel<INNER, PREC, 0, 6><<<grid, kThreads, 0, s>>>(a); break;
        case 8:  palsgd_inner_kernel<INNER, PREC, 0, 5><<<grid, kThreads, 0, s>>>(a); break;
        case 9:  palsgd_inner_kernel<INNER, PREC, 0, 8><<<grid, kThreads, 0, s>>>(a); break;
        case 13: palsgd_inner_kernel<INNER, PREC, -1, 4><<<grid, kThreads, 0, s>>>(a); break;
        case 14: palsgd_inner_kernel<INNER, PREC, -1, 3><<<grid, kThreads, 0, s>>>(a); break;
        case 15: palsgd_inner_kernel<INNER, PREC, -1, 5><<<grid, kThreads, 0, s>>>(a); break;
        default:      // measured best on B200: one 128-bit load per stream and thread, many CTAs per SM
            if (PREC) palsgd_inner_kernel<INNER, PREC, 1, 4><<<grid, kThreads, 0, s>>>(a);
            else      palsgd_inner_kernel<INNER, PREC, 1, 6><<<grid, kThreads, 0, s>>>(a);
            break;
    }
}

using PipeKernel = void (*)(const InnerArgs, uint32_t, uint32_t);
template <int INNER, int PREC, int NC>
PipeKernel pipe_kernel_ptr()
{
    if constexpr (NC == 0) return palsgd_inner_pipe_all_kernel<INNER, PREC>;
    else return palsgd_inner_pipe_kernel<INNER, PREC, NC>;
}

// Persistent TMA-ring kernel: one CTA per SM, as many stages as shared memory holds.
template <int INNER, int PREC, int NC>
int launch_inner_pipe(palsgd_ctx* ctx, const InnerArgs& a, cudaStream_t s)
{
    constexpr uint32_t stage_bytes = ((INNER == 0 ? 12u : 8u) + (PREC ? 2u : 4u)) * kStageElems;
    const int budget = ctx->smem_optin - 4096;              // static shared memory and the system's share
    int stages = std::min<int>(kPipeMaxStages, budget / (int)stage_bytes);
    if (ctx->pipe_stages > 0) stages = std::min(stages, ctx->pipe_stages);
    if (stages < 2) return PALSGD_EUNSUPPORTED;
    const size_t dyn = (size_t)stages * stage_bytes;
    auto kernel = pipe_kernel_ptr<INNER, PREC, NC>();
    constexpr unsigned threads = NC == 0 ? 1024u : (unsigned)NC + 32u;
    static int attr_for_device = -1;                         // opt in to large dynamic shared memory once
    int dev = 0;
    PALSGD_CUDA(ctx, cudaGetDevice(&dev));
    if (attr_for_device != dev) {
        PALSGD_CUDA(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, budget));
        attr_for_device = dev;
    }
    const uint64_t n_items = (uint64_t)ctx->tb.n_full * ctx->cfg.K * (ctx->chunk_elems / kStageElems);
    const int cap = ctx->grid_cap_inner > 0 ? ctx->grid_cap_inner : ctx->sm_count;
    const unsigned grid = grid_for(n_items, cap);
    return launch_checked(ctx, [&] { kernel<<<grid, threads, dyn, s>>>(a, (uint32_t)stages, stage_bytes); });
}

// NC = 0 selects the form in which all 1024 threads consume and thread 0 also produces.
template <int INNER, int PREC>
int launch_inner_pipe_nc(palsgd_ctx* ctx, int variant, const InnerArgs& a, cudaStream_t s)
{
    if (variant == 11) return launch_inner_pipe<INNER, PREC, 256>(ctx, a, s);
    if (variant == 10) return launch_inner_pipe<INNER, PREC, 512>(ctx, a, s);
    return launch_inner_pipe<INNER, PREC, 0>(ctx, a, s);
}

// Norm pass of the gradient clip: per-worker norms (ddp = false) or the norm of the averaged gradient.
int launch_gradnorm(palsgd_ctx* ctx, bool ddp, cudaStream_t s)
{
    NormArgs a{};
    a.tb = ctx->tb;
    a.seed = ctx->cfg.seed;
    a.thr = ctx->thr;
    a.max_norm = ctx->max_grad_norm;
    a.Kf = (float)ctx->cfg.K;
    a.ddp = ddp ? 1u : 0u;
    // chunks per work item: up to 8 (4 for the K-stream averaged form), fewer while that would leave
    // under ~2048 items; fixed by the problem, so results never depend on the device or on tuning knobs
    const uint32_t kitems = ddp ? 1u : ctx->cfg.K;
    const uint64_t items1 = (uint64_t)ctx->tb.n_chunks * kitems;
    a.group = (uint32_t)std::min<uint64_t>(ddp ? 4 : 8, std::max<uint64_t>(1, items1 / 2048));
    const uint64_t n_groups = (ctx->tb.n_chunks + a.group - 1) / a.group;
    const unsigned grid = grid_for(n_groups * kitems, ctx->grid_cap_inner);
    const bool bf = ctx->cfg.precision == PALSGD_PREC_BF16_MASTER;
    return launch_checked(ctx, [&] {
        if (bf) palsgd_gradnorm_kernel<1><<<grid, kThreads, 0, s>>>(a);
        else    palsgd_gradnorm_kernel<0><<<grid, kThreads, 0, s>>>(a);
    });
}

int launch_inner(palsgd_ctx* ctx, const InnerArgs& a, cudaStream_t s)
{
    // the shared-memory-ring forms do not carry the clip coefficient: clipped steps take the register path
    const bool whole_step = a.k_begin == 0 && a.k_count == ctx->cfg.K && a.tick;
    if (whole_step && !a.clip_on && ctx->inner_variant >= 10 && ctx->inner_variant <= 12 && ctx->tb.n_full > 0 &&
        ctx->chunk_elems % kStageElems == 0) {
        const bool adam_ = ctx->cfg.inner == PALSGD_INNER_ADAMW;
        const bool bf_ = ctx->cfg.precision == PALSGD_PREC_BF16_MASTER;
        const int v_ = ctx->inner_variant;
        if (adam_ && !bf_)  return launch_inner_pipe_nc<0, 0>(ctx, v_, a, s);
        if (!adam_ && !bf_) return launch_inner_pipe_nc<1, 0>(ctx, v_, a, s);
        if (adam_ && bf_)   return launch_inner_pipe_nc<0, 1>(ctx, v_, a, s);
        return launch_inner_pipe_nc<1, 1>(ctx, v_, a, s);
    }
    const uint64_t n_items = (uint64_t)ctx->tb.n_chunks * a.k_count;
    const bool adam = ctx->cfg.inner == PALSGD_INNER_ADAMW;
    const bool bf = ctx->cfg.precision == PALSGD_PREC_BF16_MASTER;
    int v = ctx->inner_variant;
    InnerArgs b = a;
    // with nothing to stream a one-CTA launch still advances the counters
    unsigned grid = grid_for(n_items, ctx->grid_cap_inner);
    // Default: a persistent grid (as many CTAs as are resident at once) that draws its work items from a queue
    // in device memory -- no tail of idle SMs, one prologue per CTA (measured +0.5 .. +6 % over one CTA per
    // item, most on small models).  Variant 18 = the default shape with one CTA per item.
    if (v == 0 && whole_step && ctx->sm_count > 0 && ctx->grid_cap_inner == 0) {
        b.dynamic = 1;
        grid = grid_for(n_items, ctx->sm_count * (bf ? 4 : 6));
    }
    if (v == 18) v = 0;
    return launch_checked(ctx, [&] {
        if (adam && !bf)       launch_inner_variant<0, 0>(v, grid, s, b);
        else if (!adam && !bf) launch_inner_variant<1, 0>(v, grid, s, b);
        else if (adam && bf)   launch_inner_variant<0, 1>(v, grid, s, b);
        else                   launch_inner_variant<1, 1>(v, grid, s, b);
    });
}

}  // namespace

// ------------------------------------------------------------------------- init

extern "C" int palsgd_init(palsgd_ctx** out, const palsgd_config* cfg, size_t n_tensors,
                           const uint64_t* numel, const palsgd_buffers* bufs, void* stream)
{
    if (!out) return PALSGD_EINVAL;
    *out = nullptr;
    int rc = validate_config(cfg);
    if (rc) return rc;
    if (n_tensors == 0 || !numel || !bufs) return PALSGD_EINVAL;
    const uint32_t K = cfg->K;
    const bool bf = cfg->precision == PALSGD_PREC_BF16_MASTER;
    const bool adam = cfg->inner == PALSGD_INNER_ADAMW;
    if (!bufs->param || !bufs->grad || !bufs->m || !bufs->global || !bufs->outer_mom) return PALSGD_EINVAL;
    if (bf && !bufs->master) return PALSGD_EINVAL;
    if (adam && !bufs->v) return PALSGD_EINVAL;
    const bool oadam = cfg->outer_opt == PALSGD_OUTER_ADAMW;
    if (oadam && !bufs->outer_v) return PALSGD_EINVAL;

    // which buffer kinds exist, and their element sizes
    const size_t ps = elem_size_param(cfg->precision);
    struct Kind { int id; size_t esize; bool present; };
    const Kind kinds[5] = {{0, ps, true}, {1, ps, true}, {2, 4, bf}, {3, 4, true}, {4, 4, adam}};

    uint64_t P = 0;
    for (size_t j = 0; j < n_tensors; ++j) {
        if (numel[j] > (1ull << 40)) return PALSGD_EINVAL;
        P += numel[j];
        for (uint32_t k = 0; k < K; ++k) {
            const size_t idx = (size_t)k * n_tensors + j;
            for (const Kind& kd : kinds) {
                if (!kd.present) continue;
                const void* p = buf_ptr(bufs, kd.id, idx);
                if (!p && numel[j] > 0) return PALSGD_EINVAL;
                if (!aligned(p, kd.esize)) return PALSGD_EALIGN;
            }
        }
        if ((!bufs->global[j] || !bufs->outer_mom[j]) && numel[j] > 0) return PALSGD_EINVAL;
        if (!aligned(bufs->global[j], 4) || !aligned(bufs->outer_mom[j], 4)) return PALSGD_EALIGN;
        if (oadam) {
            if (!bufs->outer_v[j] && numel[j] > 0) return PALSGD_EINVAL;
            if (!aligned(bufs->outer_v[j], 4)) return PALSGD_EALIGN;
        }
    }

    palsgd_ctx* ctx = new (std::nothrow) palsgd_ctx();
    if (!ctx) return PALSGD_ENOMEM;
    ctx->cfg = *cfg;
    ctx->n_tensors = n_tensors;
    ctx->numel.assign(numel, numel + n_tensors);
    ctx->P = P;
    ctx->thr = threshold_of(cfg->p);
    ctx->outer_lr = cfg->outer_lr;
    // work item of the outer kernel, measured on B200: with K + 2 streams per element few slots need
    // larger slices to amortise the per-item prologue (K = 4: 0.88 -> 0.95 of the copy rate)
    ctx->outer_sub_elems = K < 8 ? 4096u : kOuterSubElems;
    ctx->ddp_sub_elems = bf ? 4096u : kDdpSubElems;
    ctx->h_grad_dev.assign(bufs->grad, bufs->grad + (size_t)K * n_tensors);
    ctx->h_global_dev.assign(bufs->global, bufs->global + n_tensors);

    // ---- fuse tensors that are adjacent in every buffer into segments
    auto adjacent = [&](size_t j) {           // is tensor j+1 right behind tensor j everywhere?
        for (uint32_t k = 0; k < K; ++k) {
            const size_t a = (size_t)k * n_tensors + j, b = a + 1;
            for (const Kind& kd : kinds) {
                if (!kd.present) continue;
                const char* pa = static_cast<const char*>(buf_ptr(bufs, kd.id, a));
                const char* pb = static_cast<const char*>(buf_ptr(bufs, kd.id, b));
                if (pa + numel[j] * kd.esize != pb) return false;
            }
        }
        const char* ga = reinterpret_cast<const char*>(bufs->global[j]);
        const char* ua = reinterpret_cast<const char*>(bufs->outer_mom[j]);
        if (oadam && reinterpret_cast<const char*>(bufs->outer_v[j]) + numel[j] * 4 !=
                         reinterpret_cast<const char*>(bufs->outer_v[j + 1])) return false;
        return ga + numel[j] * 4 == reinterpret_cast<const char*>(bufs->global[j + 1]) &&
               ua + numel[j] * 4 == reinterpret_cast<const char*>(bufs->outer_mom[j + 1]);
    };
    for (size_t j = 0; j < n_tensors;) {
        Segment sg{j, 1, numel[j]};
        while (sg.first_tensor + sg.n_tensors < n_tensors &&
               adjacent(sg.first_tensor + sg.n_tensors - 1)) {
            sg.numel += numel[sg.first_tensor + sg.n_tensors];
            sg.n_tensors += 1;
        }
        j += sg.n_tensors;
        if (sg.numel > 0) ctx->segs.push_back(sg);
    }
    const size_t n_seg = ctx->segs.size();

    // ---- chunk table and per-segment vector-path flag
    // Elements per inner work item, measured best on B200: 4096 for fp32 AdamW, 8192 otherwise.
    ctx->chunk_elems = (!bf && adam) ? 4096u : kChunkElems;
    if (const char* e = std::getenv("PALSGD_CHUNK_ELEMS")) {      // tuning aid: a multiple of 1024
        const long v = std::atol(e);
        if (v >= 1024 && v <= (1 << 20) && v % 1024 == 0) ctx->chunk_elems = (uint32_t)v;
    }
    std::vector<Chunk> chunks;
    for (size_t s = 0; s < n_seg; ++s) {
        const Segment& sg = ctx->segs[s];
        bool vec = aligned(bufs->global[sg.first_tensor], 16) && aligned(bufs->outer_mom[sg.first_tensor], 16) &&
                   (!oadam || aligned(bufs->outer_v[sg.first_tensor], 16));
        for (uint32_t k = 0; k < K && vec; ++k)
            for (const Kind& kd : kinds)
                if (kd.present && !aligned(buf_ptr(bufs, kd.id, (size_t)k * n_tensors + sg.first_tensor), 16))
                    vec = false;
        for (uint64_t off = 0; off < sg.numel; off += ctx->chunk_elems) {
            const uint64_t len = sg.numel - off < ctx->chunk_elems ? sg.numel - off : ctx->chunk_elems;
            chunks.push_back(Chunk{off, (uint32_t)len, (uint32_t)s | (vec ? kSegVecFlag : 0u)});
        }
    }
    if (chunks.size() > 0x7FFFFFFFull / K) { delete ctx; return PALSGD_EUNSUPPORTED; }
    // full, aligned chunks first: the pipelined kernel streams exactly those through shared memory
    const uint32_t full_len = ctx->chunk_elems;
    auto is_full = [full_len](const Chunk& c) { return (c.seg & kSegVecFlag) && c.len == full_len; };
    const size_t n_full = std::stable_partition(chunks.begin(), chunks.end(), is_full) - chunks.begin();

    // ---- one device blob: [DevState][chunks][7 pointer tables]
    const size_t per_slot = (size_t)K * n_seg * sizeof(void*);
    const size_t per_seg = n_seg * sizeof(void*);
    size_t off_state = 0;
    size_t off_chunks = round_up(sizeof(DevState), 256);
    size_t off_tabs = round_up(off_chunks + chunks.size() * sizeof(Chunk), 256);
    const size_t off_norm = off_tabs + 5 * round_up(per_slot, 256) + 3 * round_up(per_seg, 256) + 256;
    const size_t total = off_norm + round_up(chunks.size() * K * sizeof(double2), 256) + 256;
    std::vector<char> host(total, 0);
    DevState hs{};
    for (uint32_t k = 0; k < kMaxWorkers; ++k) { hs.pow1[k] = 1.0; hs.pow2[k] = 1.0; hs.clip[k] = 1.f; }
    std::memcpy(host.data() + off_state, &hs, sizeof(hs));
    if (!chunks.empty()) std::memcpy(host.data() + off_chunks, chunks.data(), chunks.size() * sizeof(Chunk));

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    {
        int dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess) {
            cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, dev);
            cudaDeviceGetAttribute(&ctx->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
        }
        (void)cudaGetLastError();
    }
    if (cudaMalloc(&ctx->d_blob, total) != cudaSuccess) {
        cudaError_t e = cudaGetLastError();
        g_noctx_err = std::string("cudaMalloc: ") + cudaGetErrorString(e);
        delete ctx;
        return e == cudaErrorMemoryAllocation ? PALSGD_ENOMEM : PALSGD_ECUDA;
    }
    char* d = static_cast<char*>(ctx->d_blob);
    size_t cur = off_tabs;
    auto fill_slot_table = [&](int kind) -> void* {
        void** h = reinterpret_cast<void**>(host.data() + cur);
        for (uint32_t k = 0; k < K; ++k)
            for (size_t sgi = 0; sgi < n_seg; ++sgi)
                h[(size_t)k * n_seg + sgi] =
                    const_cast<void*>(buf_ptr(bufs, kind, (size_t)k * n_tensors + ctx->segs[sgi].first_tensor));
        void* dev = d + cur;
        cur += round_up(per_slot, 256);
        return dev;
    };
    auto fill_seg_table = [&](float* const* src) -> void* {
        void** h = reinterpret_cast<void**>(host.data() + cur);
        for (size_t sgi = 0; sgi < n_seg; ++sgi) h[sgi] = src[ctx->segs[sgi].first_tensor];
        void* dev = d + cur;
        cur += round_up(per_seg, 256);
        return dev;
    };
    Tables& tb = ctx->tb;
    tb.st = reinterpret_cast<DevState*>(d + off_state);
    tb.chunks = reinterpret_cast<const Chunk*>(d + off_chunks);
    tb.n_chunks = (uint32_t)chunks.size();
    tb.n_seg = (uint32_t)n_seg;
    tb.K = K;
    tb.n_full = (uint32_t)n_full;
    tb.chunk_elems = ctx->chunk_elems;
    void* t_param = fill_slot_table(0);
    tb.grad = static_cast<const void* const*>(fill_slot_table(1));
    void* t_master = bf ? fill_slot_table(2) : nullptr;
    tb.m = static_cast<float* const*>(fill_slot_table(3));
    tb.v = adam ? static_cast<float* const*>(fill_slot_table(4)) : nullptr;
    tb.global = static_cast<float* const*>(fill_seg_table(bufs->global));
    tb.outer_mom = static_cast<float* const*>(fill_seg_table(bufs->outer_mom));
    tb.outer_v = oadam ? static_cast<float* const*>(fill_seg_table(bufs->outer_v)) : nullptr;
    tb.xf = static_cast<float* const*>(bf ? t_master : t_param);
    tb.xw = bf ? static_cast<__nv_bfloat16* const*>(t_param) : nullptr;
    tb.norm_part = reinterpret_cast<double2*>(d + off_norm);

    cudaError_t e = cudaMemcpyAsync(ctx->d_blob, host.data(), total, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);      // `host` is pageable and dies with this scope
    if (e != cudaSuccess) { rc = cuda_fail(nullptr, e, "table upload"); cudaFree(ctx->d_blob); delete ctx; return rc; }

    if (tb.n_chunks > 0) {
        const OuterArgs oa = outer_args(ctx);
        const unsigned grid = grid_for(tb.n_chunks, 0);
        rc = launch_checked(ctx, [&] {
            if (bf) palsgd_init_kernel<1><<<grid, kThreads, 0, s>>>(oa, adam ? 1 : 0);
            else    palsgd_init_kernel<0><<<grid, kThreads, 0, s>>>(oa, adam ? 1 : 0);
        });
        if (rc) { g_noctx_err = ctx->cuda_err; cudaFree(ctx->d_blob); delete ctx; return rc; }
    }
    *out = ctx;
    return PALSGD_OK;
}

// ------------------------------------------------------------------------- steps

// Arguments of the fused inner kernel for one whole step (all K workers, counters ticked).
static InnerArgs inner_args(const palsgd_ctx* ctx, double lr_t, double eta_t)
{
    const palsgd_config& c = ctx->cfg;
    InnerArgs a{};
    a.tb = ctx->tb;
    a.seed = c.seed;
    a.thr = ctx->thr;
    a.beta1 = c.beta1;
    a.beta2 = c.beta2;
    // The coefficient of a branch that p rules out is never formed (p = 0: no pull; p = 1: no gradient step).
    const double lr_d = c.p < 1.0 ? lr_t / (1.0 - c.p) : 0.0;
    a.lr = (float)lr_d;
    a.beta_pull = c.p > 0.0 ? (float)(lr_t * eta_t / c.p) : 0.0f;
    a.b1 = (float)c.beta1;
    a.b2 = (float)c.beta2;
    a.omb1 = (float)(1.0 - c.beta1);
    a.omb2 = (float)(1.0 - c.beta2);
    a.eps = (float)c.eps;
    a.decay = (float)(1.0 - lr_d * c.weight_decay);
    a.mu = (float)c.momentum;
    a.wd = (float)c.weight_decay;
    a.chunk_major = (uint32_t)ctx->chunk_major;
    // clipped gradients: one norm pass first (not needed when every worker pulls)
    a.clip_on = (ctx->max_grad_norm > 0.0 && c.p < 1.0) ? 1u : 0u;
    a.k_begin = 0;
    a.k_count = c.K;
    a.tick = 1;
    return a;
}

extern "C" int palsgd_inner_step(palsgd_ctx* ctx, double lr_t, double eta_t, void* stream)
{
    if (!ctx) return PALSGD_EINVAL;
    if (!finite_nonneg(lr_t) || !finite_nonneg(eta_t)) return PALSGD_EINVAL;
    const InnerArgs a = inner_args(ctx, lr_t, eta_t);
    int rc = PALSGD_OK;
    if (a.clip_on) { rc = launch_gradnorm(ctx, false, static_cast<cudaStream_t>(stream)); if (rc) return rc; }
    rc = launch_inner(ctx, a, static_cast<cudaStream_t>(stream));
    if (rc) return rc;
    ctx->t += 1;
    return PALSGD_OK;
}

extern "C" int palsgd_ddp_step(palsgd_ctx* ctx, double lr_t, void* stream)
{
    if (!ctx) return PALSGD_EINVAL;
    if (!finite_nonneg(lr_t)) return PALSGD_EINVAL;
    const palsgd_config& c = ctx->cfg;
    DdpArgs a{};
    a.tb = ctx->tb;
    a.beta1 = c.beta1;
    a.beta2 = c.beta2;
    a.lr = (float)lr_t;
    a.b1 = (float)c.beta1;
    a.b2 = (float)c.beta2;
    a.omb1 = (float)(1.0 - c.beta1);
    a.omb2 = (float)(1.0 - c.beta2);
    a.eps = (float)c.eps;
    a.decay = (float)(1.0 - lr_t * c.weight_decay);
    a.mu = (float)c.momentum;
    a.wd = (float)c.weight_decay;
    a.Kf = (float)c.K;
    a.sub_elems = ctx->ddp_sub_elems;
    a.parts = (ctx->chunk_elems + a.sub_elems - 1) / a.sub_elems;
    // with nothing to stream a one-CTA launch still advances the counters
    const unsigned grid = grid_for((uint64_t)ctx->tb.n_chunks * a.parts, ctx->grid_cap_outer);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool adam = c.inner == PALSGD_INNER_ADAMW;
    const bool bf = c.precision == PALSGD_PREC_BF16_MASTER;
    a.clip_on = ctx->max_grad_norm > 0.0 ? 1u : 0u;
    int rc = PALSGD_OK;
    if (a.clip_on) { rc = launch_gradnorm(ctx, true, s); if (rc) return rc; }
    // staged form: new state in shared memory, fanned out to the K slots by bulk asynchronous stores
    const size_t stage_bytes = (size_t)a.sub_elems * ((adam ? 12u : 8u) + (bf ? 2u : 0u));
    const bool bcast = ctx->ddp_variant != 1 && (int)stage_bytes <= ctx->smem_optin - 4096;   // measured best
    using DdpKernel = void (*)(const DdpArgs);
    DdpKernel kernel;
    if (bcast) kernel = adam ? (bf ? palsgd_ddp_kernel<0, 1, 1> : palsgd_ddp_kernel<0, 0, 1>)
                             : (bf ? palsgd_ddp_kernel<1, 1, 1> : palsgd_ddp_kernel<1, 0, 1>);
    else       kernel = adam ? (bf ? palsgd_ddp_kernel<0, 1, 0> : palsgd_ddp_kernel<0, 0, 0>)
                             : (bf ? palsgd_ddp_kernel<1, 1, 0> : palsgd_ddp_kernel<1, 0, 0>);
    if (bcast && stage_bytes + 4096 > 48 * 1024)   // static + dynamic above the default limit: opt in (idempotent)
        PALSGD_CUDA(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)stage_bytes));
    unsigned g = grid;
    const int dyn = ctx->outer_dynamic < 0 ? 4 : ctx->outer_dynamic;
    if (dyn && ctx->grid_cap_outer == 0 && ctx->sm_count > 0) {                      // persistent grid + work queue
        a.dynamic = 1;
        g = grid_for((uint64_t)ctx->tb.n_chunks * a.parts, ctx->sm_count * dyn);
    }
    rc = launch_checked(ctx, [&] { kernel<<<g, kThreads, bcast ? stage_bytes : 0, s>>>(a); });
    if (rc) return rc;
    ctx->t += 1;
    return PALSGD_OK;
}

extern "C" int palsgd_pseudo_sync(palsgd_ctx* ctx, uint64_t worker_mask, double beta, void* stream)
{
    if (!ctx || !std::isfinite(beta)) return PALSGD_EINVAL;
    const uint32_t K = ctx->cfg.K;
    if (K < 64 && (worker_mask >> K) != 0) return PALSGD_EINVAL;
    if (worker_mask == 0 || ctx->tb.n_chunks == 0) return PALSGD_OK;
    PullArgs a{};
    a.tb = ctx->tb;
    a.mask = worker_mask;
    a.beta = (float)beta;
    const unsigned grid = grid_for((uint64_t)ctx->tb.n_chunks * K, ctx->grid_cap_inner);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool bf = ctx->cfg.precision == PALSGD_PREC_BF16_MASTER;
    return launch_checked(ctx, [&] {
        if (bf) palsgd_pull_kernel<1, 2><<<grid, kThreads, 0, s>>>(a);
        else    palsgd_pull_kernel<0, 4><<<grid, kThreads, 0, s>>>(a);
    });
}

extern "C" int palsgd_outer_sync(palsgd_ctx* ctx, void* stream)
{
    if (!ctx) return PALSGD_EINVAL;
    if (ctx->tb.n_chunks > 0) {
        const OuterArgs a = outer_args(ctx);
        const unsigned grid = grid_for((uint64_t)ctx->tb.n_chunks * a.parts, ctx->grid_cap_outer);
        cudaStream_t s = static_cast<cudaStream_t>(stream);
        const bool bf = ctx->cfg.precision == PALSGD_PREC_BF16_MASTER;
        const bool oadam = ctx->cfg.outer_opt == PALSGD_OUTER_ADAMW;
        // staged form: new x_g (and u, bf16 copy) in shared memory, K slots written by bulk asynchronous stores
        const size_t stage_bytes = (size_t)a.sub_elems * (8u + (oadam ? 4u : 0u) + (bf ? 2u : 0u));
        const bool bcast = ctx->outer_variant != 1 && (int)stage_bytes <= ctx->smem_optin - 4096;   // measured best
        using OuterKernel = void (*)(const OuterArgs);
        OuterKernel kernel;
        if (bcast) kernel = bf ? (oadam ? palsgd_outer_kernel<1, 1, 1> : palsgd_outer_kernel<1, 0, 1>)
                               : (oadam ? palsgd_outer_kernel<0, 1, 1> : palsgd_outer_kernel<0, 0, 1>);
        else       kernel = bf ? (oadam ? palsgd_outer_kernel<1, 1, 0> : palsgd_outer_kernel<1, 0, 0>)
                               : (oadam ? palsgd_outer_kernel<0, 1, 0> : palsgd_outer_kernel<0, 0, 0>);
        if (bcast && stage_bytes + 4096 > 48 * 1024)
            PALSGD_CUDA(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)stage_bytes));
        OuterArgs b = a;
        unsigned g = grid;
        const int dyn = ctx->outer_dynamic < 0 ? 0 : ctx->outer_dynamic;
        if (dyn && ctx->grid_cap_outer == 0 && ctx->sm_count > 0) {                  // persistent grid + work queue
            b.dynamic = 1;
            g = grid_for((uint64_t)ctx->tb.n_chunks * a.parts, ctx->sm_count * dyn);
        }
        int rc = launch_checked(ctx, [&] { kernel<<<g, kThreads, bcast ? stage_bytes : 0, s>>>(b); });
        if (rc) return rc;
    }
    if (ctx->cfg.outer_opt == PALSGD_OUTER_ADAMW) {
        ctx->opow1 *= ctx->cfg.outer_beta1;
        ctx->opow2 *= ctx->cfg.outer_beta2;
    }
    ctx->n_outer += 1;
    return PALSGD_OK;
}

extern "C" int palsgd_step(palsgd_ctx* ctx, double lr_t, double eta_t, void* stream)
{
    int rc = palsgd_inner_step(ctx, lr_t, eta_t, stream);
    if (rc) return rc;
    if (ctx->t % ctx->cfg.H == 0) rc = palsgd_outer_sync(ctx, stream);
    return rc;
}

// ------------------------------------------------------------------------- captured cycle

extern "C" int palsgd_cycle_capture(palsgd_ctx* ctx, double lr_t, double eta_t)
{
    if (!ctx) return PALSGD_EINVAL;
    if (!finite_nonneg(lr_t) || !finite_nonneg(eta_t)) return PALSGD_EINVAL;
    if (ctx->t % ctx->cfg.H != 0) return PALSGD_ESTATE;             // a cycle starts right after a sync
    if (ctx->cfg.outer_opt == PALSGD_OUTER_ADAMW) return PALSGD_EUNSUPPORTED;   // its scalars change every round
    if (ctx->cfg.H > (1u << 16)) return PALSGD_EUNSUPPORTED;
    if (ctx->cycle_exec) { cudaGraphExecDestroy(ctx->cycle_exec); ctx->cycle_exec = nullptr; }

    // Capture on a stream of our own (the caller's may be the legacy default stream, which cannot capture).
    // Nothing runs during capture, so the host mirrors are put back afterwards.
    const uint64_t t0 = ctx->t, n0 = ctx->n_outer, l0 = ctx->launches;
    cudaStream_t cs = nullptr;
    PALSGD_CUDA(ctx, cudaStreamCreateWithFlags(&cs, cudaStreamNonBlocking));
    cudaError_t e = cudaStreamBeginCapture(cs, cudaStreamCaptureModeThreadLocal);
    int rc = PALSGD_OK;
    if (e == cudaSuccess) {
        for (uint64_t i = 0; i < ctx->cfg.H && rc == PALSGD_OK; ++i) rc = palsgd_step(ctx, lr_t, eta_t, cs);
        cudaGraph_t graph = nullptr;
        e = cudaStreamEndCapture(cs, &graph);                       // also ends a capture that failed midway
        if (rc == PALSGD_OK && e == cudaSuccess) e = cudaGraphInstantiate(&ctx->cycle_exec, graph, 0);
        if (graph) cudaGraphDestroy(graph);
    }
    ctx->cycle_launches = ctx->launches - l0;
    ctx->t = t0; ctx->n_outer = n0; ctx->launches = l0;
    cudaStreamDestroy(cs);
    if (rc == PALSGD_OK && e != cudaSuccess) rc = cuda_fail(ctx, e, "cycle capture");
    if (rc != PALSGD_OK && ctx->cycle_exec) { cudaGraphExecDestroy(ctx->cycle_exec); ctx->cycle_exec = nullptr; }
    if (rc != PALSGD_OK) (void)cudaGetLastError();
    return rc;
}

extern "C" int palsgd_cycle_launch(palsgd_ctx* ctx, void* stream)
{
    if (!ctx) return PALSGD_EINVAL;
    if (!ctx->cycle_exec || ctx->t % ctx->cfg.H != 0) return PALSGD_ESTATE;
    PALSGD_CUDA(ctx, cudaGraphLaunch(ctx->cycle_exec, static_cast<cudaStream_t>(stream)));
    ctx->t += ctx->cfg.H;
    ctx->n_outer += 1;
    ctx->launches += ctx->cycle_launches;
    return PALSGD_OK;
}

extern "C" int palsgd_step_host(palsgd_ctx* ctx, const void* const* h_grad, double lr_t, double eta_t,
                                float* const* h_global, uint8_t* h_decisions, int* synced, void* stream)
{
    if (!ctx || !h_grad) return PALSGD_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t n = ctx->n_tensors;
    const size_t gs = elem_size_param(ctx->cfg.precision);
    if (!finite_nonneg(lr_t) || !finite_nonneg(eta_t)) return PALSGD_EINVAL;
    const uint32_t K = ctx->cfg.K;
    for (uint32_t k = 0; k < K; ++k) {                       // a pulling worker's pointers are not looked at
        if (draw_pull(ctx->cfg.seed, ctx->t, k, ctx->thr)) continue;
        for (size_t j = 0; j < n; ++j)
            if (!h_grad[(size_t)k * n + j] && ctx->numel[j] > 0) return PALSGD_EINVAL;
    }
    // host -> device gradients of worker k; tensors adjacent on both sides travel as one copy.
    // A worker that pulls in this step has no use for a gradient (Algorithm 1 takes one branch or the
    // other), so nothing is transferred for it.
    auto copy_worker = [&](uint32_t k, cudaStream_t cs) -> int {
        if (draw_pull(ctx->cfg.seed, ctx->t, k, ctx->thr)) return PALSGD_OK;
        for (const Segment& sg : ctx->segs) {
            size_t j = sg.first_tensor;
            const size_t end = sg.first_tensor + sg.n_tensors;
            while (j < end) {
                const size_t idx = (size_t)k * n + j;
                const char* src = static_cast<const char*>(h_grad[idx]);
                size_t bytes = ctx->numel[j] * gs;
                size_t j2 = j + 1;
                while (j2 < end && static_cast<const char*>(h_grad[(size_t)k * n + j2]) == src + bytes) {
                    bytes += ctx->numel[j2] * gs;
                    ++j2;
                }
                if (bytes)
                    PALSGD_CUDA(ctx, cudaMemcpyAsync(const_cast<void*>(ctx->h_grad_dev[idx]), src, bytes,
                                                     cudaMemcpyHostToDevice, cs));
                j = j2;
            }
        }
        return PALSGD_OK;
    };
    InnerArgs a = inner_args(ctx, lr_t, eta_t);
    int rc = PALSGD_OK;
    if (K > 1 && !a.clip_on) {
        // Worker by worker: the copies run on a stream of the library's own, and the part of the step that
        // needs worker k's gradient is launched as soon as that gradient has arrived, so the arithmetic
        // hides behind the transfer of the following workers.  The last launch ticks the counters.
        if (!ctx->copy_stream) {
            PALSGD_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
            PALSGD_CUDA(ctx, cudaEventCreateWithFlags(&ctx->copy_may_start, cudaEventDisableTiming));
            ctx->copy_done.resize(K, nullptr);
            for (uint32_t k = 0; k < K; ++k)
                PALSGD_CUDA(ctx, cudaEventCreateWithFlags(&ctx->copy_done[k], cudaEventDisableTiming));
        }
        PALSGD_CUDA(ctx, cudaEventRecord(ctx->copy_may_start, s));          // earlier readers of the gradients
        PALSGD_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_stream, ctx->copy_may_start, 0));
        for (uint32_t k = 0; k < K; ++k) {
            rc = copy_worker(k, ctx->copy_stream);
            if (rc) return rc;
            PALSGD_CUDA(ctx, cudaEventRecord(ctx->copy_done[k], ctx->copy_stream));
        }
        for (uint32_t k = 0; k < K; ++k) {
            PALSGD_CUDA(ctx, cudaStreamWaitEvent(s, ctx->copy_done[k], 0));
            a.k_begin = k;
            a.k_count = 1;
            a.tick = k + 1 == K ? 1u : 0u;
            rc = launch_inner(ctx, a, s);
            if (rc) return rc;
        }
        ctx->t += 1;
    } else {
        for (uint32_t k = 0; k < K; ++k) { rc = copy_worker(k, s); if (rc) return rc; }
        rc = palsgd_inner_step(ctx, lr_t, eta_t, stream);
        if (rc) return rc;
    }
    const bool sync_now = ctx->t % ctx->cfg.H == 0;
    if (sync_now) { rc = palsgd_outer_sync(ctx, stream); if (rc) return rc; }
    if (synced) *synced = sync_now ? 1 : 0;
    if (h_decisions)
        PALSGD_CUDA(ctx, cudaMemcpyAsync(h_decisions, ctx->tb.st->last_b, ctx->cfg.K, cudaMemcpyDeviceToHost, s));
    if (sync_now && h_global) {
        for (const Segment& sg : ctx->segs) {
            size_t j = sg.first_tensor;
            const size_t end = sg.first_tensor + sg.n_tensors;
            while (j < end) {
                char* dst = reinterpret_cast<char*>(h_global[j]);
                if (!dst) return PALSGD_EINVAL;
                size_t bytes = ctx->numel[j] * 4;
                size_t j2 = j + 1;
                while (j2 < end && reinterpret_cast<char*>(h_global[j2]) == dst + bytes) {
                    bytes += ctx->numel[j2] * 4;
                    ++j2;
                }
                if (bytes)
                    PALSGD_CUDA(ctx, cudaMemcpyAsync(dst, ctx->h_global_dev[j], bytes, cudaMemcpyDeviceToHost, s));
                j = j2;
            }
        }
    }
    PALSGD_CUDA(ctx, cudaStreamSynchronize(s));
    return PALSGD_OK;
}

// ------------------------------------------------------------------------- counters

extern "C" int palsgd_get_counters(palsgd_ctx* ctx, uint64_t* t, uint64_t* s_k, uint64_t* n_outer,
                                   uint8_t* last_b, void* stream)
{
    if (!ctx) return PALSGD_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    DevState hs;
    PALSGD_CUDA(ctx, cudaMemcpyAsync(&hs, ctx->tb.st, sizeof(hs), cudaMemcpyDeviceToHost, s));
    PALSGD_CUDA(ctx, cudaStreamSynchronize(s));
    if (t) *t = hs.t;
    if (n_outer) *n_outer = ctx->n_outer;
    for (uint32_t k = 0; k < ctx->cfg.K; ++k) {
        if (s_k) s_k[k] = hs.s[k];
        if (last_b) last_b[k] = hs.last_b[k];
    }
    if (hs.error != 0) return PALSGD_ETIMEOUT;
    return hs.t == ctx->t ? PALSGD_OK : PALSGD_ESTATE;
}

extern "C" int palsgd_set_counters(palsgd_ctx* ctx, uint64_t t, const uint64_t* s_k, uint64_t n_outer,
                                   void* stream)
{
    if (!ctx || !s_k) return PALSGD_EINVAL;
    for (uint32_t k = 0; k < ctx->cfg.K; ++k)
        if (s_k[k] > t) return PALSGD_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    DevState hs{};
    hs.t = t;
    for (uint32_t k = 0; k < kMaxWorkers; ++k) {
        hs.pow1[k] = 1.0; hs.pow2[k] = 1.0; hs.clip[k] = 1.f;
        if (k < ctx->cfg.K) {
            hs.s[k] = s_k[k];
            for (uint64_t i = 0; i < s_k[k]; ++i) {      // the same running products the kernels form
                hs.pow1[k] *= ctx->cfg.beta1;
                hs.pow2[k] *= ctx->cfg.beta2;
                if (hs.pow1[k] == 0.0 && hs.pow2[k] == 0.0) break;
            }
        }
    }
    PALSGD_CUDA(ctx, cudaMemcpyAsync(ctx->tb.st, &hs, sizeof(hs), cudaMemcpyHostToDevice, s));
    PALSGD_CUDA(ctx, cudaStreamSynchronize(s));          // hs lives on this stack frame
    ctx->t = t;
    ctx->n_outer = n_outer;
    ctx->opow1 = ctx->opow2 = 1.0;
    if (ctx->cfg.outer_opt == PALSGD_OUTER_ADAMW)
        for (uint64_t i = 0; i < n_outer; ++i) {             // the running products of n_outer syncs
            ctx->opow1 *= ctx->cfg.outer_beta1;
            ctx->opow2 *= ctx->cfg.outer_beta2;
            if (ctx->opow1 == 0.0 && ctx->opow2 == 0.0) break;
        }
    return PALSGD_OK;
}

extern "C" int palsgd_set_outer_lr(palsgd_ctx* ctx, double outer_lr)
{
    if (!ctx || !std::isfinite(outer_lr)) return PALSGD_EINVAL;
    ctx->outer_lr = outer_lr;
    return PALSGD_OK;
}

extern "C" double palsgd_schedule_value(int kind, uint64_t t, uint64_t warmup, uint64_t total, double base,
                                        double min_value, double start_factor)
{
    if ((kind != PALSGD_SCHED_WARMUP_CONSTANT && kind != PALSGD_SCHED_WARMUP_COSINE) || !std::isfinite(base) ||
        !std::isfinite(min_value) || !std::isfinite(start_factor))
        return std::nan("");
    if (t < warmup) return base * (start_factor + (1.0 - start_factor) * (double)t / (double)warmup);
    if (kind == PALSGD_SCHED_WARMUP_CONSTANT || total <= warmup) return base;
    const double kPi = 3.14159265358979323846;
    const double tau = (double)((t < total ? t : total) - warmup);
    return min_value + (base - min_value) * (1.0 + std::cos(kPi * tau / (double)(total - warmup))) / 2.0;
}

extern "C" int palsgd_set_grad_clip(palsgd_ctx* ctx, double max_norm)
{
    if (!ctx || !(max_norm >= 0.0) || !std::isfinite(max_norm)) return PALSGD_EINVAL;
    ctx->max_grad_norm = max_norm;
    return PALSGD_OK;
}

extern "C" int palsgd_get_grad_norms(palsgd_ctx* ctx, double* sumsq, float* clip, void* stream)
{
    if (!ctx) return PALSGD_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    DevState hs;
    PALSGD_CUDA(ctx, cudaMemcpyAsync(&hs, ctx->tb.st, sizeof(hs), cudaMemcpyDeviceToHost, s));
    PALSGD_CUDA(ctx, cudaStreamSynchronize(s));
    for (uint32_t k = 0; k < ctx->cfg.K; ++k) {
        if (sumsq) sumsq[k] = hs.sumsq[k];
        if (clip) clip[k] = hs.clip[k];
    }
    return PALSGD_OK;
}

extern "C" int palsgd_get_launch_count(palsgd_ctx* ctx, uint64_t* n_launches)
{
    if (!ctx || !n_launches) return PALSGD_EINVAL;
    *n_launches = ctx->launches;
    return PALSGD_OK;
}

extern "C" int palsgd_set_tuning(palsgd_ctx* ctx, int knob, int64_t value)
{
    if (!ctx || value < 0 || value > 0x7FFFFFFF) return PALSGD_EINVAL;
    switch (knob) {
        case PALSGD_TUNE_INNER_GRID_CAP: ctx->grid_cap_inner = (int)value; return PALSGD_OK;
        case PALSGD_TUNE_OUTER_GRID_CAP: ctx->grid_cap_outer = (int)value; return PALSGD_OK;
        case PALSGD_TUNE_INNER_VARIANT:  ctx->inner_variant = (int)value; return PALSGD_OK;
        case PALSGD_TUNE_PIPE_STAGES:    ctx->pipe_stages = (int)value; return PALSGD_OK;
        case PALSGD_TUNE_CHUNK_MAJOR:    ctx->chunk_major = value != 0; return PALSGD_OK;
        case PALSGD_TUNE_OUTER_SUB_ELEMS:
            if (value < 1024 || value % 1024 != 0) return PALSGD_EINVAL;
            ctx->outer_sub_elems = (uint32_t)value;
            return PALSGD_OK;
        case PALSGD_TUNE_OUTER_DYNAMIC:
            if (value > 32) return PALSGD_EINVAL;
            ctx->outer_dynamic = (int)value;
            return PALSGD_OK;
        case PALSGD_TUNE_OUTER_VARIANT:
            if (value > 2) return PALSGD_EINVAL;
            ctx->outer_variant = (int)value;
            return PALSGD_OK;
        case PALSGD_TUNE_DDP_VARIANT:
            if (value > 2) return PALSGD_EINVAL;
            ctx->ddp_variant = (int)value;
            return PALSGD_OK;
        case PALSGD_TUNE_DDP_SUB_ELEMS:
            if (value < 1024 || value % 1024 != 0) return PALSGD_EINVAL;
            ctx->ddp_sub_elems = (uint32_t)value;
            return PALSGD_OK;
        default: return PALSGD_EINVAL;
    }
}

// ------------------------------------------------------------------------- pure host helpers

extern "C" int palsgd_decision(uint64_t seed, uint64_t t, uint32_t k, double p)
{
    if (!(p >= 0.0 && p <= 1.0) || k >= PALSGD_MAX_WORKERS) return PALSGD_EINVAL;
    return draw_pull(seed, t, k, threshold_of(p)) ? 1 : 0;
}

extern "C" const char* palsgd_strerror(int status)
{
    switch (status) {
        case PALSGD_OK: return "ok";
        case PALSGD_EINVAL: return "invalid argument";
        case PALSGD_EALIGN: return "pointer not aligned to its element size";
        case PALSGD_ECUDA: return "CUDA error";
        case PALSGD_ESTATE: return "call not valid in this state";
        case PALSGD_ENOMEM: return "out of memory";
        case PALSGD_EUNSUPPORTED: return "unsupported combination";
        case PALSGD_ETIMEOUT: return "a bounded device-side wait expired";
        case PALSGD_ETOOBIG: return "tensor list exceeds the fixed scratch of the no-allocation entry point";
        default: return "unknown status";
    }
}

extern "C" const char* palsgd_last_cuda_error(palsgd_ctx* ctx)
{
    return ctx ? ctx->cuda_err.c_str() : g_noctx_err.c_str();
}

extern "C" void palsgd_destroy(palsgd_ctx* ctx)
{
    if (!ctx) return;
    if (ctx->cycle_exec) cudaGraphExecDestroy(ctx->cycle_exec);
    for (cudaEvent_t e : ctx->copy_done) if (e) cudaEventDestroy(e);
    if (ctx->copy_may_start) cudaEventDestroy(ctx->copy_may_start);
    if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
    if (ctx->d_blob) cudaFree(ctx->d_blob);
    delete ctx;
}
