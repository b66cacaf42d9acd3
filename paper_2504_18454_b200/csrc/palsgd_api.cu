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
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "palsgd_kernels.cuh"
#include "palsgd_norm.cuh"

using namespace palsgd;

// Default launch shapes of the outer-sync and DDP kernels (CTAs per SM of a persistent grid that draws
// its items from a queue; 0 = one CTA per item), measured on B200.
// A CTA that handles several items alternates between two stage buffers when both fit in this many bytes
// (beyond it the second buffer would cost resident CTAs, which measured far worse than a drained stage).
constexpr size_t kTwoStageLimit = 32 * 1024;
constexpr int kOuterCtasPerSm = 0;
constexpr int kDdpCtasPerSm = 4;

// palsgd_step_host: one small host -> device copy that a kernel performs (see palsgd_gather_host_kernel).
struct HostCopy {
    const unsigned char* src;     // pinned host memory, through its device alias; 16-byte aligned
    unsigned char*       dst;     // device memory, 16-byte aligned
    uint64_t             bytes;
};
// Copies below this size go through the gather kernel when a worker has at least kGatherMinCopies of them.
constexpr size_t kGatherMaxBytes = 2 * 1024 * 1024;    // measured: 256 KB, 1 MB and 16 MB all do worse on the three model-shaped lists
constexpr size_t kGatherMinCopies = 8;
constexpr size_t kGatherItemBytes = 32 * 1024;               // longer copies are cut into table entries of this size

// The many small tensors of a framework-style layout (biases, normalisation scales: a few KB each) cost a copy
// engine several microseconds apiece, whatever their size.  This kernel performs all of a worker's small copies
// in one launch: every CTA takes whole entries of the table and reads the PINNED host memory directly (the
// table itself lives there too).  Large tensors still travel through the copy engine.
__global__ void __launch_bounds__(256) palsgd_gather_host_kernel(const HostCopy* __restrict__ items, uint32_t n_items)
{
    for (uint32_t it = blockIdx.x; it < n_items; it += gridDim.x) {
        const HostCopy c = items[it];
        const uint32_t n16 = (uint32_t)(c.bytes >> 4);       // (an entry is at most kGatherItemBytes long)
        const uint4* __restrict__ s = reinterpret_cast<const uint4*>(c.src);
        uint4* __restrict__ d = reinterpret_cast<uint4*>(c.dst);
        uint32_t i = threadIdx.x;
        for (; i + 3 * 256 < n16; i += 4 * 256) {            // four reads of host memory in flight per thread
            const uint4 a0 = s[i], a1 = s[i + 256], a2 = s[i + 512], a3 = s[i + 768];
            d[i] = a0; d[i + 256] = a1; d[i + 512] = a2; d[i + 768] = a3;
        }
        for (; i < n16; i += 256) d[i] = s[i];
        for (uint32_t j = (n16 << 4) + threadIdx.x; j < c.bytes; j += 256) c.dst[j] = c.src[j];
    }
}

struct Segment {
    size_t   first_tensor;
    size_t   n_tensors;
    uint64_t numel;
    int      head;     // elements to peel off the front so that what follows is aligned (16 bytes at least) in every
                       // buffer (0..255); -1 = no such count exists: the whole segment takes the scalar path
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
    // item tables of the outer-sync and DDP kernels (their own allocations: a tuning knob may rebuild them)
    Chunk* d_oitems = nullptr;  uint32_t n_oitems = 0;
    Chunk* d_ditems = nullptr;  uint32_t n_ditems = 0;
    uint64_t P = 0;
    uint64_t exch_numel = 0;                 // floats in the exchange buffer of the multi-GPU outer sync
    uint32_t k0 = 0;                         // the decision stream's index of local worker 0
    // host mirrors
    uint64_t t = 0, n_outer = 0, launches = 0;
    uint64_t thr = 0;
    int grid_cap_inner = 0, grid_cap_outer = 0;   // 0 = one CTA per work item
    int inner_variant = 0;                        // 0 = persistent grid + work queue (default), 18 = one CTA per item
    uint32_t chunk_elems = kChunkElems;           // elements per chunk-table entry (fixed at init)
    uint32_t outer_sub_elems = kOuterSubElems;    // elements per work item of the outer kernel
    uint32_t ddp_sub_elems = kDdpSubElems;        // elements per work item of the DDP warm-up kernel
    int ddp_variant = 0;                          // 0 = default, 1 = per-thread stores, 2 = staged bulk stores
    int outer_variant = 0;                        // the same for the outer kernel
    int outer_dynamic = -1;                       // outer / DDP kernels: CTAs per SM of a persistent grid, 0 = one CTA
                                                  // per item, -1 = default (kOuterCtasPerSm / kDdpCtasPerSm)
    double max_grad_norm = 0.0;                   // global-norm clip threshold, 0 = off
    double outer_lr = 0.0;                        // OuterOPT learning rate of the next sync
    double opow1 = 1.0, opow2 = 1.0;              // outer_beta^n_outer (AdamW as OuterOPT), running products
    cudaStream_t copy_stream = nullptr;           // palsgd_step_host: host -> device copies run here ...
    std::vector<cudaEvent_t> copy_done;           // ... and signal worker k's gradient with copy_done[k]
    cudaEvent_t copy_may_start = nullptr;         // recorded on the caller's stream before the copies begin
    HostCopy* gather_items = nullptr;             // pinned host table of the small copies of one palsgd_step_host call
    size_t gather_cap = 0;                        //   (read by palsgd_gather_host_kernel straight from host memory)
    cudaGraphExec_t cycle_exec = nullptr;         // captured H-step cycle (palsgd_cycle_capture) or nullptr
    uint64_t cycle_launches = 0;                  // kernels inside one captured cycle
    int sm_count = 0, smem_optin = 0;             // device attributes read at init
    int device = 0;                               // the device that was current at palsgd_init
    bool failed = false;                          // a CUDA call failed midway through an earlier entry point:
                                                  // device state and host mirrors may disagree, so every later
                                                  // call that would touch them returns PALSGD_ESTATE
    std::string cuda_err;
};

namespace {

thread_local std::string g_noctx_err;

int cuda_fail(palsgd_ctx* ctx, cudaError_t e, const char* what)
{
    std::string msg = std::string(what) + ": " + cudaGetErrorString(e);
    if (ctx) { ctx->cuda_err = msg; ctx->failed = true; } else g_noctx_err = msg;
    return PALSGD_ECUDA;
}

#define PALSGD_CUDA(ctx, call)                                            \
    do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return cuda_fail((ctx), e_, #call); } while (0)

// Entry points that read or advance the state refuse a context that an earlier CUDA failure left half-advanced.
#define PALSGD_USABLE(ctx)                                                \
    do { if (!(ctx)) return PALSGD_EINVAL; if ((ctx)->failed) return PALSGD_ESTATE; } while (0)

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

// Cut every segment into pieces of at most `piece` elements (a multiple of 1024).  A segment whose
// buffers all become 16-byte aligned after `head` elements gets those elements as one scalar piece
// and vector pieces behind it; full vector pieces are listed first (the small ones fill the tail of
// a launch instead of sitting between large ones).
std::vector<Chunk> cut_segments(const std::vector<Segment>& segs, uint32_t piece)
{
    std::vector<Chunk> out;
    for (size_t s = 0; s < segs.size(); ++s) {
        const Segment& sg = segs[s];
        uint64_t off = 0;
        const bool vec = sg.head >= 0;
        if (sg.head > 0) {
            off = std::min<uint64_t>((uint64_t)sg.head, sg.numel);
            out.push_back(Chunk{0, (uint32_t)off, (uint32_t)s});
        }
        for (; off < sg.numel; off += piece) {
            const uint64_t len = std::min<uint64_t>(sg.numel - off, piece);
            out.push_back(Chunk{off, (uint32_t)len, (uint32_t)s | (vec ? kSegVecFlag : 0u)});
        }
    }
    auto is_full = [piece](const Chunk& c) { return (c.seg & kSegVecFlag) && c.len == piece; };
    std::stable_partition(out.begin(), out.end(), is_full);
    return out;
}

// (Re)build one of the item tables on the device.  Synchronous; frees the previous table.
int upload_items(palsgd_ctx* ctx, const std::vector<Chunk>& items, Chunk** d_items, uint32_t* n_items)
{
    if (*d_items) { PALSGD_CUDA(ctx, cudaDeviceSynchronize()); cudaFree(*d_items); *d_items = nullptr; }
    *n_items = (uint32_t)items.size();
    if (items.empty()) return PALSGD_OK;
    PALSGD_CUDA(ctx, cudaMalloc(reinterpret_cast<void**>(d_items), items.size() * sizeof(Chunk)));
    PALSGD_CUDA(ctx, cudaMemcpy(*d_items, items.data(), items.size() * sizeof(Chunk), cudaMemcpyHostToDevice));
    return PALSGD_OK;
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
    a.items = ctx->d_oitems;
    a.n_items = ctx->n_oitems;
    a.sub_elems = ctx->outer_sub_elems;
    a.n_stage = 1;
    return a;
}

// Raise a kernel's dynamic-shared-memory limit when a launch needs more than the limit in force.  The
// attribute belongs to the function on a device, not to a context: the limits set so far are kept per
// (device, kernel) for the whole process and only ever raised, so that contexts with different item sizes
// cannot lower each other's limit, and the runtime call is made once instead of on every launch.
int ensure_dyn_smem(palsgd_ctx* ctx, const void* kernel, size_t bytes)
{
    if (bytes + 4096 <= 48 * 1024) return PALSGD_OK;         // static + dynamic within the default limit
    struct Entry { int dev; const void* kernel; int bytes; };
    static std::mutex mu;
    static std::vector<Entry> limits;
    std::lock_guard<std::mutex> lock(mu);
    for (Entry& e : limits)
        if (e.dev == ctx->device && e.kernel == kernel) {
            if (e.bytes >= (int)bytes) return PALSGD_OK;
            PALSGD_CUDA(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
            e.bytes = (int)bytes;
            return PALSGD_OK;
        }
    PALSGD_CUDA(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
    limits.push_back(Entry{ctx->device, kernel, (int)bytes});
    return PALSGD_OK;
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
    a.k0 = ctx->k0;
    // chunks per group (the unit a CTA fetches at a time): up to 8 (4 for the K-stream averaged form), fewer
    // while that would leave under ~2048 groups
    const uint32_t kitems = ddp ? 1u : ctx->cfg.K;
    const uint64_t items1 = (uint64_t)ctx->tb.n_chunks * kitems;
    a.group = (uint32_t)std::min<uint64_t>(ddp ? 4 : 8, std::max<uint64_t>(1, items1 / 2048));
    const uint64_t n_groups = (ctx->tb.n_chunks + a.group - 1) / a.group;
    // a persistent grid: every CTA works for one worker and leaves one partial (3 CTAs per SM are resident)
    int cap = ctx->sm_count > 0 ? ctx->sm_count * 3 : 444;
    if (ctx->grid_cap_inner > 0) cap = std::min(cap, ctx->grid_cap_inner);
    // (at least one CTA per worker, whatever the cap: a CTA serves a single worker)
    const unsigned grid = std::max<unsigned>(grid_for(n_groups * kitems, cap), kitems);
    const bool bf = ctx->cfg.precision == PALSGD_PREC_BF16_MASTER;
    return launch_checked(ctx, [&] {
        if (bf) { if (ddp) palsgd_gradnorm_kernel<1, 1><<<grid, kThreads, 0, s>>>(a);
                  else     palsgd_gradnorm_kernel<1, 0><<<grid, kThreads, 0, s>>>(a); }
        else    { if (ddp) palsgd_gradnorm_kernel<0, 1><<<grid, kThreads, 0, s>>>(a);
                  else     palsgd_gradnorm_kernel<0, 0><<<grid, kThreads, 0, s>>>(a); }
    });
}

// Launch shape of the fused inner kernel, measured on B200: one 128-bit load per stream and thread,
// registers held to 4 (mixed precision) or 6 (fp32) CTAs per SM.
int launch_inner(palsgd_ctx* ctx, const InnerArgs& a, cudaStream_t s)
{
    const bool whole_step = a.k_begin == 0 && a.k_count == ctx->cfg.K && a.tick;
    const uint64_t n_items = (uint64_t)ctx->tb.n_chunks * a.k_count;
    const bool adam = ctx->cfg.inner == PALSGD_INNER_ADAMW;
    const bool bf = ctx->cfg.precision == PALSGD_PREC_BF16_MASTER;
    InnerArgs b = a;
    // with nothing to stream a one-CTA launch still advances the counters
    unsigned grid = grid_for(n_items, ctx->grid_cap_inner);
    // Default: a persistent grid (as many CTAs as are resident at once) that draws its work items from a queue
    // in device memory -- no tail of idle SMs, one prologue per CTA (measured +0.5 .. +6 % over one CTA per
    // item, most on small models).  Variant 18 = the same shape with one CTA per item.
    if (ctx->inner_variant != 18 && whole_step && ctx->sm_count > 0 && ctx->grid_cap_inner == 0) {
        b.dynamic = 1;
        grid = grid_for(n_items, ctx->sm_count * (bf ? 4 : 6));
    }
    return launch_checked(ctx, [&] {
        if (adam && !bf)       palsgd_inner_kernel<0, 0, 1, 6><<<grid, kThreads, 0, s>>>(b);
        else if (!adam && !bf) palsgd_inner_kernel<1, 0, 1, 6><<<grid, kThreads, 0, s>>>(b);
        else if (adam && bf)   palsgd_inner_kernel<0, 1, 1, 4><<<grid, kThreads, 0, s>>>(b);
        else                   palsgd_inner_kernel<1, 1, 1, 4><<<grid, kThreads, 0, s>>>(b);
    });
}

// Host-only planning of a tensor list: argument checks, fusion of adjacent tensors into segments, the
// alignment head of every segment.  Looks at the ADDRESSES in `bufs` only, never at what they point to.
int plan_segments(const palsgd_config* cfg, size_t n_tensors, const uint64_t* numel, const palsgd_buffers* bufs,
                  std::vector<Segment>& segs, uint64_t& P)
{
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

    P = 0;
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
    // Elements to peel off a segment's front so that what follows is aligned in every buffer.  Needed
    // by the vector paths and the bulk stores: 16 bytes.  Wanted: a multiple of 256 elements (1024
    // bytes of fp32, 512 of bf16).  Measured on packed lists shifted by s elements: the inner kernel
    // runs at its full rate for s = 256, 1.5 % under it for s = 128, 3-5 % under it for any s below
    // that, 16-byte aligned or not.  So: the smallest h that puts every fp32 buffer on 1024 bytes and
    // every bf16 buffer on 512, else on 512 and 256, else on 256 and 128, else all on 16: 0 for buffers
    // that are aligned already, 255 for a packed list shifted by one element, 7 or less when the
    // buffers' offsets differ.  -1 if no h gives even 16 bytes.
    auto head_of = [&](size_t first) {
        auto all_aligned = [&](int h, size_t a4, size_t a2) {    // bytes wanted: 4-byte kinds, 2-byte kinds
            if (!aligned(reinterpret_cast<const char*>(bufs->global[first]) + 4 * h, a4) ||
                !aligned(reinterpret_cast<const char*>(bufs->outer_mom[first]) + 4 * h, a4) ||
                (oadam && !aligned(reinterpret_cast<const char*>(bufs->outer_v[first]) + 4 * h, a4)))
                return false;
            for (uint32_t k = 0; k < K; ++k)
                for (const Kind& kd : kinds)
                    if (kd.present && !aligned(static_cast<const char*>(buf_ptr(bufs, kd.id, (size_t)k * n_tensors + first)) +
                                                   kd.esize * h, kd.esize == 4 ? a4 : a2))
                        return false;
            return true;
        };
        const size_t want[4][2] = {{1024, 512}, {512, 256}, {256, 128}, {16, 16}};
        for (const auto& w : want)
            for (int h = 0; h < (int)(w[1] / 2); ++h)
                if (all_aligned(h, w[0], w[1])) return h;
        return -1;
    };
    for (size_t j = 0; j < n_tensors;) {
        Segment sg{j, 1, numel[j], 0};
        while (sg.first_tensor + sg.n_tensors < n_tensors &&
               adjacent(sg.first_tensor + sg.n_tensors - 1)) {
            sg.numel += numel[sg.first_tensor + sg.n_tensors];
            sg.n_tensors += 1;
        }
        j += sg.n_tensors;
        // (an empty tensor between two adjacent ones is skipped over by the fusion above; the first
        //  tensor of a non-empty segment may itself be empty, its pointer still marks the start)
        if (sg.numel > 0) { sg.head = head_of(sg.first_tensor); segs.push_back(sg); }
    }
    return PALSGD_OK;
}

// Elements per inner work item, measured best on B200: 4096 for fp32 AdamW, 8192 otherwise.
inline uint32_t chunk_elems_for(const palsgd_config& cfg)
{
    return (cfg.precision != PALSGD_PREC_BF16_MASTER && cfg.inner == PALSGD_INNER_ADAMW) ? 4096u : kChunkElems;
}

}  // namespace

// ------------------------------------------------------------------------- init

extern "C" int palsgd_init(palsgd_ctx** out, const palsgd_config* cfg, size_t n_tensors,
                           const uint64_t* numel, const palsgd_buffers* bufs, void* stream)
{
    if (!out) return PALSGD_EINVAL;
    *out = nullptr;
    std::vector<Segment> planned;
    uint64_t P = 0;
    int rc = plan_segments(cfg, n_tensors, numel, bufs, planned, P);
    if (rc) return rc;
    const uint32_t K = cfg->K;
    const bool bf = cfg->precision == PALSGD_PREC_BF16_MASTER;
    const bool adam = cfg->inner == PALSGD_INNER_ADAMW;
    const bool oadam = cfg->outer_opt == PALSGD_OUTER_ADAMW;

    palsgd_ctx* ctx = new (std::nothrow) palsgd_ctx();
    if (!ctx) return PALSGD_ENOMEM;
    ctx->cfg = *cfg;
    ctx->n_tensors = n_tensors;
    ctx->numel.assign(numel, numel + n_tensors);
    ctx->P = P;
    ctx->thr = threshold_of(cfg->p);
    ctx->outer_lr = cfg->outer_lr;
    // work item of the outer kernel, measured on B200: 1024 elements; for K = 5..7 (K + 2 streams per element,
    // 4 CTAs per SM) larger items amortise the per-item prologue; K <= 4 runs the narrow-batch form of the
    // kernel with 5 CTAs per SM, which does best with the small item (2048 for K <= 2)
    ctx->outer_sub_elems = (K > 4 && K < 8) ? 4096u : K <= 2 ? 2048u : kOuterSubElems;
    ctx->ddp_sub_elems = kDdpSubElems;
    ctx->h_grad_dev.assign(bufs->grad, bufs->grad + (size_t)K * n_tensors);
    ctx->h_global_dev.assign(bufs->global, bufs->global + n_tensors);

    ctx->segs = std::move(planned);
    const size_t n_seg = ctx->segs.size();

    // ---- chunk table of the inner kernel; item tables of the outer-sync and DDP kernels
    ctx->chunk_elems = chunk_elems_for(*cfg);
    const std::vector<Chunk> chunks = cut_segments(ctx->segs, ctx->chunk_elems);
    const std::vector<Chunk> oitems = cut_segments(ctx->segs, ctx->outer_sub_elems);
    const std::vector<Chunk> ditems = cut_segments(ctx->segs, ctx->ddp_sub_elems);
    if (chunks.size() > 0x7FFFFFFFull / K || oitems.size() > 0x7FFFFFFFull || ditems.size() > 0x7FFFFFFFull) {
        delete ctx;
        return PALSGD_EUNSUPPORTED;
    }

    // ---- one device blob: [DevState][chunks][7 pointer tables]
    const size_t per_slot = (size_t)K * n_seg * sizeof(void*);
    const size_t per_seg = n_seg * sizeof(void*);
    size_t off_state = 0;
    size_t off_chunks = round_up(sizeof(DevState), 256);
    size_t off_tabs = round_up(off_chunks + chunks.size() * sizeof(Chunk), 256);
    const size_t off_norm = off_tabs + 5 * round_up(per_slot, 256) + 4 * round_up(per_seg, 256) + 256;
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
            ctx->device = dev;
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
    {   // exchange-buffer offsets: the buffer is the tensor list packed back to back (a function of the
        // element counts alone, so that every GPU of a job lays it out alike whatever its memory layout)
        uint64_t* h = reinterpret_cast<uint64_t*>(host.data() + cur);
        std::vector<uint64_t> prefix(n_tensors + 1, 0);
        for (size_t j = 0; j < n_tensors; ++j) prefix[j + 1] = prefix[j] + numel[j];
        for (size_t sgi = 0; sgi < n_seg; ++sgi) h[sgi] = prefix[ctx->segs[sgi].first_tensor];
        ctx->exch_numel = P;
        tb.exch_off = reinterpret_cast<const uint64_t*>(d + cur);
        cur += round_up(per_seg, 256);
    }
    tb.norm_part = reinterpret_cast<double2*>(d + off_norm);

    cudaError_t e = cudaMemcpyAsync(ctx->d_blob, host.data(), total, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);      // `host` is pageable and dies with this scope
    if (e != cudaSuccess) { rc = cuda_fail(nullptr, e, "table upload"); cudaFree(ctx->d_blob); delete ctx; return rc; }
    rc = upload_items(ctx, oitems, &ctx->d_oitems, &ctx->n_oitems);
    if (rc == PALSGD_OK) rc = upload_items(ctx, ditems, &ctx->d_ditems, &ctx->n_ditems);
    if (rc) { g_noctx_err = ctx->cuda_err; palsgd_destroy(ctx); return rc == PALSGD_ECUDA ? rc : PALSGD_ENOMEM; }

    if (tb.n_chunks > 0) {
        const OuterArgs oa = outer_args(ctx);
        const unsigned grid = grid_for(tb.n_chunks, 0);
        rc = launch_checked(ctx, [&] {
            if (bf) palsgd_init_kernel<1><<<grid, kThreads, 0, s>>>(oa, adam ? 1 : 0);
            else    palsgd_init_kernel<0><<<grid, kThreads, 0, s>>>(oa, adam ? 1 : 0);
        });
        if (rc) { g_noctx_err = ctx->cuda_err; palsgd_destroy(ctx); return rc; }
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
    // clipped gradients: one norm pass first (not needed when every worker pulls)
    a.clip_on = (ctx->max_grad_norm > 0.0 && c.p < 1.0) ? 1u : 0u;
    a.k_begin = 0;
    a.k_count = c.K;
    a.k0 = ctx->k0;
    a.tick = 1;
    return a;
}

extern "C" int palsgd_inner_step(palsgd_ctx* ctx, double lr_t, double eta_t, void* stream)
{
    PALSGD_USABLE(ctx);
    if (!finite_nonneg(lr_t) || !finite_nonneg(eta_t)) return PALSGD_EINVAL;
    const InnerArgs a = inner_args(ctx, lr_t, eta_t);
    int rc = PALSGD_OK;
    if (a.clip_on) { rc = launch_gradnorm(ctx, false, static_cast<cudaStream_t>(stream)); if (rc) return rc; }
    rc = launch_inner(ctx, a, static_cast<cudaStream_t>(stream));
    if (rc) return rc;
    ctx->t += 1;
    return PALSGD_OK;
}

// One DDP warm-up step.  sum_in == nullptr: the K local gradients are averaged in the kernel; otherwise the
// gradient sum over all K_total workers of the job is read from the exchange buffer.
static int ddp_launch(palsgd_ctx* ctx, double lr_t, void* stream, const float* sum_in, uint32_t K_total)
{
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
    a.Kf = (float)K_total;
    a.sum_in = sum_in;
    a.items = ctx->d_ditems;
    a.n_items = ctx->n_ditems;
    a.sub_elems = ctx->ddp_sub_elems;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool adam = c.inner == PALSGD_INNER_ADAMW;
    const bool bf = c.precision == PALSGD_PREC_BF16_MASTER;
    a.clip_on = ctx->max_grad_norm > 0.0 ? 1u : 0u;
    int rc = PALSGD_OK;
    if (a.clip_on) { rc = launch_gradnorm(ctx, true, s); if (rc) return rc; }
    // with nothing to stream a one-CTA launch still advances the counters
    unsigned grid = grid_for(a.n_items, ctx->grid_cap_outer);
    const int dyn = ctx->outer_dynamic < 0 ? kDdpCtasPerSm : ctx->outer_dynamic;
    if (dyn && ctx->grid_cap_outer == 0 && ctx->sm_count > 0) {                      // persistent grid + work queue
        a.dynamic = 1;
        grid = grid_for(a.n_items, ctx->sm_count * dyn);
    }
    // staged form: new state in shared memory, fanned out to the K slots by bulk asynchronous stores; a CTA
    // that handles several items alternates between two stage buffers
    const size_t one_stage = (size_t)a.sub_elems * ((adam ? 12u : 8u) + (bf ? 2u : 0u));
    a.n_stage = (grid < a.n_items && 2 * one_stage <= kTwoStageLimit) ? 2u : 1u;
    const size_t stage_bytes = one_stage * a.n_stage;
    const bool bcast = ctx->ddp_variant != 1 && (int)stage_bytes <= ctx->smem_optin - 4096;   // measured best
    using DdpKernel = void (*)(const DdpArgs);
    DdpKernel kernel;
    if (sum_in) {
        if (!bcast) return PALSGD_EUNSUPPORTED;               // the exchange form exists in the staged form only
        kernel = adam ? (bf ? palsgd_ddp_kernel<0, 1, 1, 1> : palsgd_ddp_kernel<0, 0, 1, 1>)
                      : (bf ? palsgd_ddp_kernel<1, 1, 1, 1> : palsgd_ddp_kernel<1, 0, 1, 1>);
    } else if (bcast) kernel = adam ? (bf ? palsgd_ddp_kernel<0, 1, 1> : palsgd_ddp_kernel<0, 0, 1>)
                                    : (bf ? palsgd_ddp_kernel<1, 1, 1> : palsgd_ddp_kernel<1, 0, 1>);
    else              kernel = adam ? (bf ? palsgd_ddp_kernel<0, 1, 0> : palsgd_ddp_kernel<0, 0, 0>)
                                    : (bf ? palsgd_ddp_kernel<1, 1, 0> : palsgd_ddp_kernel<1, 0, 0>);
    if (bcast) { rc = ensure_dyn_smem(ctx, reinterpret_cast<const void*>(kernel), stage_bytes); if (rc) return rc; }
    rc = launch_checked(ctx, [&] { kernel<<<grid, kThreads, bcast ? stage_bytes : 0, s>>>(a); });
    if (rc) return rc;
    ctx->t += 1;
    return PALSGD_OK;
}

extern "C" int palsgd_ddp_step(palsgd_ctx* ctx, double lr_t, void* stream)
{
    PALSGD_USABLE(ctx);
    if (!finite_nonneg(lr_t)) return PALSGD_EINVAL;
    return ddp_launch(ctx, lr_t, stream, nullptr, ctx->cfg.K);
}

extern "C" int palsgd_ddp_partial(palsgd_ctx* ctx, float* exchange, void* stream)
{
    PALSGD_USABLE(ctx);
    if (!exchange && ctx->exch_numel > 0) return PALSGD_EINVAL;
    if (!aligned(exchange, 16)) return PALSGD_EALIGN;
    if (ctx->tb.n_chunks == 0) return PALSGD_OK;
    DdpArgs a{};
    a.tb = ctx->tb;
    a.items = ctx->tb.chunks;                               // nothing is staged: the inner kernel's larger pieces serve
    a.n_items = ctx->tb.n_chunks;
    a.sum_out = exchange;
    const unsigned grid = grid_for(a.n_items, ctx->grid_cap_outer);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool bf = ctx->cfg.precision == PALSGD_PREC_BF16_MASTER;
    return launch_checked(ctx, [&] {
        if (bf) palsgd_ddp_partial_kernel<1><<<grid, kThreads, 0, s>>>(a);
        else    palsgd_ddp_partial_kernel<0><<<grid, kThreads, 0, s>>>(a);
    });
}

extern "C" int palsgd_ddp_finish(palsgd_ctx* ctx, const float* exchange, uint32_t K_total, double lr_t, void* stream)
{
    PALSGD_USABLE(ctx);
    if (!finite_nonneg(lr_t) || K_total < ctx->cfg.K) return PALSGD_EINVAL;
    if (!exchange) return PALSGD_EINVAL;
    if (!aligned(exchange, 16)) return PALSGD_EALIGN;
    if (ctx->max_grad_norm > 0.0) return PALSGD_EUNSUPPORTED;  // the norm of a gradient that lives in the exchange buffer
    return ddp_launch(ctx, lr_t, stream, exchange, K_total);
}

extern "C" int palsgd_pseudo_sync(palsgd_ctx* ctx, uint64_t worker_mask, double beta, void* stream)
{
    PALSGD_USABLE(ctx);
    if (!std::isfinite(beta)) return PALSGD_EINVAL;
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
    PALSGD_USABLE(ctx);
    if (ctx->n_oitems > 0) {
        OuterArgs a = outer_args(ctx);
        cudaStream_t s = static_cast<cudaStream_t>(stream);
        const bool bf = ctx->cfg.precision == PALSGD_PREC_BF16_MASTER;
        const bool oadam = ctx->cfg.outer_opt == PALSGD_OUTER_ADAMW;
        unsigned grid = grid_for(a.n_items, ctx->grid_cap_outer);
        const int dyn = ctx->outer_dynamic < 0 ? kOuterCtasPerSm : ctx->outer_dynamic;
        if (dyn && ctx->grid_cap_outer == 0 && ctx->sm_count > 0) {                  // persistent grid + work queue
            a.dynamic = 1;
            grid = grid_for(a.n_items, ctx->sm_count * dyn);
        }
        // staged form: new x_g (and u, bf16 copy) in shared memory, K slots written by bulk asynchronous stores;
        // a CTA that handles several items alternates between two stage buffers
        const size_t one_stage = (size_t)a.sub_elems * (8u + (oadam ? 4u : 0u) + (bf ? 2u : 0u));
        a.n_stage = (grid < a.n_items && 2 * one_stage <= kTwoStageLimit) ? 2u : 1u;
        const size_t stage_bytes = one_stage * a.n_stage;
        const bool bcast = ctx->outer_variant != 1 && (int)stage_bytes <= ctx->smem_optin - 4096;   // measured best
        using OuterKernel = void (*)(const OuterArgs);
        OuterKernel kernel;
        const bool few = ctx->cfg.K <= 4;                      // narrower load batches, one more CTA per SM
        if (bcast) kernel = bf ? (oadam ? palsgd_outer_kernel<1, 1, 1> : few ? palsgd_outer_kernel<1, 0, 1, 0, 4> : palsgd_outer_kernel<1, 0, 1>)
                               : (oadam ? palsgd_outer_kernel<0, 1, 1> : few ? palsgd_outer_kernel<0, 0, 1, 0, 4> : palsgd_outer_kernel<0, 0, 1>);
        else       kernel = bf ? (oadam ? palsgd_outer_kernel<1, 1, 0> : palsgd_outer_kernel<1, 0, 0>)
                               : (oadam ? palsgd_outer_kernel<0, 1, 0> : palsgd_outer_kernel<0, 0, 0>);
        if (bcast) { const int rc = ensure_dyn_smem(ctx, reinterpret_cast<const void*>(kernel), stage_bytes); if (rc) return rc; }
        int rc = launch_checked(ctx, [&] { kernel<<<grid, kThreads, bcast ? stage_bytes : 0, s>>>(a); });
        if (rc) return rc;
    }
    if (ctx->cfg.outer_opt == PALSGD_OUTER_ADAMW) {
        ctx->opow1 *= ctx->cfg.outer_beta1;
        ctx->opow2 *= ctx->cfg.outer_beta2;
    }
    ctx->n_outer += 1;
    return PALSGD_OK;
}

// ------------------------------------------------------------------------- outer sync over several GPUs

extern "C" int palsgd_exchange_numel(palsgd_ctx* ctx, uint64_t* n_floats)
{
    if (!ctx || !n_floats) return PALSGD_EINVAL;
    *n_floats = ctx->exch_numel;
    return PALSGD_OK;
}

extern "C" int palsgd_set_worker_offset(palsgd_ctx* ctx, uint32_t k0)
{
    PALSGD_USABLE(ctx);
    if ((uint64_t)k0 + ctx->cfg.K > 0xFFFFFFFFull) return PALSGD_EINVAL;
    ctx->k0 = k0;
    return PALSGD_OK;
}

extern "C" int palsgd_outer_partial(palsgd_ctx* ctx, float* exchange, void* stream)
{
    PALSGD_USABLE(ctx);
    if (!exchange && ctx->exch_numel > 0) return PALSGD_EINVAL;
    if (!aligned(exchange, 16)) return PALSGD_EALIGN;
    if (ctx->tb.n_chunks == 0) return PALSGD_OK;
    OuterArgs a = outer_args(ctx);
    a.sum_out = exchange;
    // nothing is staged here, so the larger pieces of the inner kernel's chunk table serve: the per-item
    // set-up (two barriers, K pointers) is paid once per 4096 or 8192 elements instead of once per 1024
    a.items = ctx->tb.chunks;
    a.n_items = ctx->tb.n_chunks;
    const unsigned grid = grid_for(a.n_items, ctx->grid_cap_outer);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return launch_checked(ctx, [&] { palsgd_outer_partial_kernel<8><<<grid, kThreads, 0, s>>>(a); });
}

extern "C" int palsgd_global_from_exchange(palsgd_ctx* ctx, const float* exchange, uint32_t K_total, void* stream)
{
    PALSGD_USABLE(ctx);
    if (K_total < ctx->cfg.K) return PALSGD_EINVAL;
    if (!exchange && ctx->exch_numel > 0) return PALSGD_EINVAL;
    if (!aligned(exchange, 16)) return PALSGD_EALIGN;
    if (ctx->n_oitems == 0) return PALSGD_OK;
    OuterArgs a = outer_args(ctx);
    a.sum_in = exchange;
    a.Kf = (float)K_total;
    const unsigned grid = grid_for(a.n_items, ctx->grid_cap_outer);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return launch_checked(ctx, [&] { palsgd_global_from_sum_kernel<0><<<grid, kThreads, 0, s>>>(a); });
}

extern "C" int palsgd_outer_finish(palsgd_ctx* ctx, const float* exchange, uint32_t K_total, void* stream)
{
    PALSGD_USABLE(ctx);
    if (K_total < ctx->cfg.K) return PALSGD_EINVAL;
    if (!exchange && ctx->exch_numel > 0) return PALSGD_EINVAL;
    if (!aligned(exchange, 16)) return PALSGD_EALIGN;
    if (ctx->n_oitems > 0) {
        OuterArgs a = outer_args(ctx);
        a.sum_in = exchange;
        a.Kf = (float)K_total;
        cudaStream_t s = static_cast<cudaStream_t>(stream);
        const bool bf = ctx->cfg.precision == PALSGD_PREC_BF16_MASTER;
        const bool oadam = ctx->cfg.outer_opt == PALSGD_OUTER_ADAMW;
        const unsigned grid = grid_for(a.n_items, ctx->grid_cap_outer);
        const size_t one_stage = (size_t)a.sub_elems * (8u + (oadam ? 4u : 0u) + (bf ? 2u : 0u));
        a.n_stage = (grid < a.n_items && 2 * one_stage <= kTwoStageLimit) ? 2u : 1u;
        const size_t stage_bytes = one_stage * a.n_stage;
        if ((int)stage_bytes > ctx->smem_optin - 4096) return PALSGD_EUNSUPPORTED;   // an item size set far too large
        using OuterKernel = void (*)(const OuterArgs);
        OuterKernel kernel = bf ? (oadam ? palsgd_outer_kernel<1, 1, 1, 1> : palsgd_outer_kernel<1, 0, 1, 1>)
                                : (oadam ? palsgd_outer_kernel<0, 1, 1, 1> : palsgd_outer_kernel<0, 0, 1, 1>);
        int rc = ensure_dyn_smem(ctx, reinterpret_cast<const void*>(kernel), stage_bytes);
        if (rc) return rc;
        rc = launch_checked(ctx, [&] { kernel<<<grid, kThreads, stage_bytes, s>>>(a); });
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
    PALSGD_USABLE(ctx);
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
    PALSGD_USABLE(ctx);
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
    PALSGD_USABLE(ctx);
    if (!h_grad) return PALSGD_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t n = ctx->n_tensors;
    const size_t gs = elem_size_param(ctx->cfg.precision);
    if (!finite_nonneg(lr_t) || !finite_nonneg(eta_t)) return PALSGD_EINVAL;
    const uint32_t K = ctx->cfg.K;
    for (uint32_t k = 0; k < K; ++k) {                       // a pulling worker's pointers are not looked at
        if (draw_pull(ctx->cfg.seed, ctx->t, ctx->k0 + k, ctx->thr)) continue;
        for (size_t j = 0; j < n; ++j)
            if (!h_grad[(size_t)k * n + j] && ctx->numel[j] > 0) return PALSGD_EINVAL;
    }
    // everything is checked before the first enqueue: the global model is read back only on a sync step
    const bool will_sync = (ctx->t + 1) % ctx->cfg.H == 0;
    if (will_sync && h_global)
        for (size_t j = 0; j < n; ++j)
            if (!h_global[j] && ctx->numel[j] > 0) return PALSGD_EINVAL;
    // host -> device gradients of worker k; tensors adjacent on both sides travel as one copy.
    // A worker that pulls in this step has no use for a gradient (Algorithm 1 takes one branch or the
    // other), so nothing is transferred for it.
    // Small copies (under kGatherMaxBytes, both ends 16-byte aligned, the source pinned) are collected and, if a
    // worker has kGatherMinCopies or more of them, performed by one launch of the gather kernel on the same stream.
    std::vector<HostCopy> small, pieces;
    std::vector<const unsigned char*> alias;
    size_t gather_used = 0;                                  // entries of the pinned table taken by earlier workers
    auto copy_worker = [&](uint32_t k, cudaStream_t cs) -> int {
        if (draw_pull(ctx->cfg.seed, ctx->t, ctx->k0 + k, ctx->thr)) return PALSGD_OK;
        small.clear();
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
                void* dst = const_cast<void*>(ctx->h_grad_dev[idx]);
                if (bytes && bytes < kGatherMaxBytes && aligned(src, 16) && aligned(dst, 16)) {
                    small.push_back(HostCopy{reinterpret_cast<const unsigned char*>(src),
                                             static_cast<unsigned char*>(dst), bytes});
                } else if (bytes)
                    PALSGD_CUDA(ctx, cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, cs));
                j = j2;
            }
        }
        // the kernel may only read memory the device can reach: every source is looked up (pinned or not, and
        // its device alias) on every call -- a buffer may have been replaced since the last one
        bool gather = small.size() >= kGatherMinCopies;
        alias.assign(small.size(), nullptr);                 // the sources as the device addresses them
        for (size_t i = 0; gather && i < small.size(); ++i) {
            cudaPointerAttributes at{};
            if (cudaPointerGetAttributes(&at, small[i].src) != cudaSuccess) { (void)cudaGetLastError(); gather = false; break; }
            if (at.type != cudaMemoryTypeHost || !at.devicePointer) { gather = false; break; }
            // the whole range must lie inside the same registration: the last byte is looked up as well
            cudaPointerAttributes at_end{};
            if (cudaPointerGetAttributes(&at_end, small[i].src + small[i].bytes - 1) != cudaSuccess ||
                at_end.type != cudaMemoryTypeHost) { (void)cudaGetLastError(); gather = false; break; }
            alias[i] = static_cast<const unsigned char*>(at.devicePointer);
        }
        if (gather) {                                        // cut into table entries of at most kGatherItemBytes
            pieces.clear();
            for (size_t i = 0; i < small.size(); ++i)
                for (uint64_t off = 0; off < small[i].bytes; off += kGatherItemBytes)
                    pieces.push_back(HostCopy{alias[i] + off, small[i].dst + off,
                                              std::min<uint64_t>(kGatherItemBytes, small[i].bytes - off)});
        }
        if (gather) {
            const size_t need = gather_used + pieces.size();
            if (need > ctx->gather_cap) {
                // grow the pinned table; earlier workers' launches of this call still read the old one
                if (gather_used > 0) PALSGD_CUDA(ctx, cudaStreamSynchronize(cs));
                HostCopy* bigger = nullptr;
                const size_t cap = std::max(need, (size_t)K * pieces.size()) + 64;
                if (cudaHostAlloc(reinterpret_cast<void**>(&bigger), cap * sizeof(HostCopy), cudaHostAllocDefault) != cudaSuccess) {
                    (void)cudaGetLastError();
                    gather = false;                          // no table: the copy engine takes them
                } else {
                    if (ctx->gather_items) cudaFreeHost(ctx->gather_items);
                    ctx->gather_items = bigger;
                    ctx->gather_cap = cap;
                    gather_used = 0;
                }
            }
        }
        if (gather) {
            HostCopy* table = ctx->gather_items + gather_used;
            std::memcpy(table, pieces.data(), pieces.size() * sizeof(HostCopy));
            gather_used += pieces.size();
            void* table_dev = nullptr;
            PALSGD_CUDA(ctx, cudaHostGetDevicePointer(&table_dev, table, 0));
            const uint32_t n_items = (uint32_t)pieces.size();
            const unsigned grid = grid_for(n_items, ctx->sm_count > 0 ? ctx->sm_count * 8 : 1184);
            return launch_checked(ctx, [&] {
                palsgd_gather_host_kernel<<<grid, 256, 0, cs>>>(static_cast<const HostCopy*>(table_dev), n_items);
            });
        }
        for (const HostCopy& c : small)
            PALSGD_CUDA(ctx, cudaMemcpyAsync(c.dst, c.src, c.bytes, cudaMemcpyHostToDevice, cs));
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
    PALSGD_USABLE(ctx);
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
    return hs.t == ctx->t ? PALSGD_OK : PALSGD_ESTATE;
}

extern "C" int palsgd_set_counters(palsgd_ctx* ctx, uint64_t t, const uint64_t* s_k, uint64_t n_outer,
                                   void* stream)
{
    PALSGD_USABLE(ctx);
    if (!s_k) return PALSGD_EINVAL;
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
    PALSGD_USABLE(ctx);
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

extern "C" int palsgd_plan_layout(const palsgd_config* cfg, size_t n_tensors, const uint64_t* numel,
                                  const palsgd_buffers* bufs, uint64_t* n_segments, uint64_t* n_chunks,
                                  uint32_t* chunk_elems, uint64_t* seg_first_tensor, uint64_t* seg_n_tensors,
                                  int32_t* seg_head)
{
    std::vector<Segment> segs;
    uint64_t P = 0;
    const int rc = plan_segments(cfg, n_tensors, numel, bufs, segs, P);
    if (rc) return rc;
    const uint32_t ce = chunk_elems_for(*cfg);
    if (n_segments) *n_segments = segs.size();
    if (n_chunks) *n_chunks = cut_segments(segs, ce).size();
    if (chunk_elems) *chunk_elems = ce;
    for (size_t i = 0; i < segs.size(); ++i) {
        if (seg_first_tensor) seg_first_tensor[i] = segs[i].first_tensor;
        if (seg_n_tensors) seg_n_tensors[i] = segs[i].n_tensors;
        if (seg_head) seg_head[i] = segs[i].head;
    }
    return PALSGD_OK;
}

extern "C" int palsgd_get_layout(palsgd_ctx* ctx, uint64_t* n_segments, uint64_t* n_chunks, uint32_t* chunk_elems)
{
    if (!ctx) return PALSGD_EINVAL;
    if (n_segments) *n_segments = ctx->segs.size();
    if (n_chunks) *n_chunks = ctx->tb.n_chunks;
    if (chunk_elems) *chunk_elems = ctx->chunk_elems;
    return PALSGD_OK;
}

extern "C" int palsgd_set_tuning(palsgd_ctx* ctx, int knob, int64_t value)
{
    if (!ctx || value < 0 || value > 0x7FFFFFFF) return PALSGD_EINVAL;
    // a recorded cycle holds the launch shapes (and item-table addresses) of the moment it was captured
    if (ctx->cycle_exec) { cudaGraphExecDestroy(ctx->cycle_exec); ctx->cycle_exec = nullptr; }
    switch (knob) {
        case PALSGD_TUNE_INNER_GRID_CAP: ctx->grid_cap_inner = (int)value; return PALSGD_OK;
        case PALSGD_TUNE_OUTER_GRID_CAP: ctx->grid_cap_outer = (int)value; return PALSGD_OK;
        case PALSGD_TUNE_INNER_VARIANT:
            if (value != 0 && value != 18) return PALSGD_EINVAL;
            ctx->inner_variant = (int)value;
            return PALSGD_OK;
        case PALSGD_TUNE_OUTER_SUB_ELEMS:
            if (value < 1024 || value % 1024 != 0 || value > (1 << 20)) return PALSGD_EINVAL;
            if (ctx->failed) return PALSGD_ESTATE;
            ctx->outer_sub_elems = (uint32_t)value;
            return upload_items(ctx, cut_segments(ctx->segs, ctx->outer_sub_elems), &ctx->d_oitems, &ctx->n_oitems);
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
            if (value < 1024 || value % 1024 != 0 || value > (1 << 20)) return PALSGD_EINVAL;
            if (ctx->failed) return PALSGD_ESTATE;
            ctx->ddp_sub_elems = (uint32_t)value;
            return upload_items(ctx, cut_segments(ctx->segs, ctx->ddp_sub_elems), &ctx->d_ditems, &ctx->n_ditems);
        default: return PALSGD_EINVAL;
    }
}

// ------------------------------------------------------------------------- pure host helpers

extern "C" int palsgd_decision(uint64_t seed, uint64_t t, uint32_t k, double p)
{
    if (!(p >= 0.0 && p <= 1.0)) return PALSGD_EINVAL;
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
    if (ctx->gather_items) cudaFreeHost(ctx->gather_items);
    if (ctx->d_oitems) cudaFree(ctx->d_oitems);
    if (ctx->d_ditems) cudaFree(ctx->d_ditems);
    if (ctx->d_blob) cudaFree(ctx->d_blob);
    delete ctx;
}
