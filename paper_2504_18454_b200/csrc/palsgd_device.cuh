// Device-side data structures shared by the PALSGD kernels and the host controller.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace palsgd {

constexpr uint32_t kMaxWorkers  = 64;      // K <= 64 (worker masks are 64-bit)
constexpr uint32_t kThreads     = 256;     // threads per CTA of every kernel here
constexpr uint32_t kChunkElems  = 8192;    // default elements per chunk-table entry = one work item of the
                                           // inner kernel (large: amortises the per-CTA prologue and tick)
constexpr uint32_t kOuterSubElems = 1024;  // default work item of the outer kernel for K >= 8 (small: K+2
                                           // streams per element need many CTAs in flight)
constexpr uint32_t kDdpSubElems = 1024;    // default work item of the DDP warm-up kernel (two stage buffers fit)
constexpr uint32_t kSegVecFlag  = 0x80000000u;   // Chunk::seg bit: 16-byte vector path allowed

// One work unit of the multi-tensor launch: `len` consecutive elements of
// segment `seg` starting at element `off`.  A segment is a maximal run of the
// caller's tensors that are adjacent in memory in every buffer.  The same
// record serves the chunk table of the inner kernel and the (finer) item
// tables of the outer-sync and DDP kernels.
struct Chunk {
    uint64_t off;
    uint32_t len;
    uint32_t seg;        // segment index | kSegVecFlag
};

// Device-resident counters: the kernels read them and the last CTA of an inner
// step advances them, so that a sequence of steps needs no host interaction
// (and can be captured in a CUDA graph).
struct DevState {
    unsigned long long t;                    // completed inner steps (Algorithm 1's t)
    unsigned long long s[kMaxWorkers];       // gradient steps taken by worker k
    double             pow1[kMaxWorkers];    // beta1^s_k  (running product, binary64)
    double             pow2[kMaxWorkers];    // beta2^s_k
    unsigned int       queue;                // next work item of a launch that hands items out dynamically
    unsigned int       done;                 // CTAs that finished the current inner launch
    unsigned int       pad0_;
    unsigned char      last_b[kMaxWorkers];  // decisions of the latest inner step
    // global-norm gradient clipping (written by the norm kernel, read by the step kernels)
    unsigned int       done_norm;            // CTAs that finished the current norm launch
    unsigned int       pad_;
    double             sumsq[kMaxWorkers];   // sum of squares of worker k's latest gradient
    float              clip[kMaxWorkers];    // coefficient that gradient is scaled by (<= 1)
};

// Device pointer tables, indexed [k * n_seg + seg] (per-slot) or [seg].
struct Tables {
    const Chunk*        chunks;
    uint32_t            n_chunks;
    uint32_t            n_seg;
    uint32_t            K;
    uint32_t            chunk_elems; // elements of a full chunk
    float* const*       xf;         // fp32 model of slot k: params (FP32) or master (BF16_MASTER)
    __nv_bfloat16* const* xw;       // bf16 working params (BF16_MASTER) else nullptr
    const void* const*  grad;       // float or bf16 gradients
    float* const*       m;
    float* const*       v;          // nullptr table entries for SGD
    float* const*       global;     // [n_seg]
    float* const*       outer_mom;  // [n_seg]
    float* const*       outer_v;    // [n_seg] second outer moment (AdamW as OuterOPT) or nullptr
    const uint64_t*     exch_off;   // [n_seg] element offset of the segment inside the exchange buffer
    DevState*           st;
    double2*            norm_part;  // [n_chunks * K] per-work-item partial sums of squares (hi, lo)
};

struct InnerArgs {
    Tables   tb;
    uint64_t seed;
    uint64_t thr;          // floor(p * 2^32): pull iff Philox word < thr
    double   beta1, beta2; // binary64 decay rates for the running products
    float    lr;           // fl32(alpha_t / (1 - p))
    float    beta_pull;    // fl32(alpha_t * eta_t / p)
    float    b1, b2, omb1, omb2, eps, decay;   // AdamW scalars, each rounded once from binary64
    float    mu, wd;       // momentum SGD scalars
    uint32_t clip_on;      // 1: scale worker k's gradient by DevState::clip[k]
    uint32_t k_begin;      // this launch covers workers k_begin .. k_begin + k_count - 1 (default: all K)
    uint32_t k_count;
    uint32_t k0;           // the decision stream's index of local worker 0 (workers spread over several contexts)
    uint32_t tick;         // 1: the last CTA advances the device counters (the launch that completes a step)
    uint32_t dynamic;      // 1: a persistent grid takes work items from DevState::queue (needs tick = 1)
};

struct PullArgs {
    Tables   tb;
    uint64_t mask;         // workers to pull
    float    beta;
};

struct OuterArgs {
    Tables tb;
    const Chunk* items;    // work items: pieces of at most sub_elems elements of a segment
    uint32_t n_items;
    float  mu, lr, Kf;
    int    nesterov;
    float  ob1, ob2, oomb1, oomb2, obc1, obc2, odecay, oeps;   // AdamW as OuterOPT (step n_outer + 1)
    uint32_t sub_elems;    // largest work item (a multiple of 4 * kThreads): size of a stage array
    uint32_t n_stage;      // stage buffers in dynamic shared memory: 2 for a persistent grid, else 1
    uint32_t dynamic;      // 1: a persistent grid takes work items from DevState::queue
    const float* sum_in;   // SUMIN kernels: the exchange buffer holding the sum over ALL workers' models
    float*       sum_out;  // partial-sum kernel: the exchange buffer that receives the local workers' sum
};

// DDP warm-up step: averaged gradient, one optimizer step taken on worker 0's state, written to all.
struct DdpArgs {
    Tables   tb;
    double   beta1, beta2; // binary64 decay rates for the running products
    float    lr;           // fl32(alpha_t): no 1/(1-p) rescaling in this phase
    float    b1, b2, omb1, omb2, eps, decay;
    float    mu, wd;
    float    Kf;
    const Chunk* items;    // work items: pieces of at most sub_elems elements of a segment
    uint32_t n_items;
    uint32_t sub_elems;    // largest work item (a multiple of 4 * kThreads): size of a stage array
    uint32_t n_stage;      // stage buffers in dynamic shared memory: 2 for a persistent grid, else 1
    uint32_t clip_on;      // 1: scale the averaged gradient by DevState::clip[0]
    uint32_t dynamic;      // 1: a persistent grid takes work items from DevState::queue
    const float* sum_in;   // SUMIN kernels: the exchange buffer holding the gradient sum over ALL workers
    float*       sum_out;  // partial-sum kernel: the exchange buffer that receives the local workers' sum
};

// Gradient-norm pass of the global-norm clip.
struct NormArgs {
    Tables   tb;
    uint64_t seed;
    uint64_t thr;          // decision threshold: workers that pull this step are skipped
    double   max_norm;     // clip threshold
    float    Kf;
    uint32_t k0;           // the decision stream's index of local worker 0
    uint32_t group;        // consecutive chunks per work item (a function of the problem size only)
};

}  // namespace palsgd
