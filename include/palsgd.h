/*
 * palsgd.h -- C ABI of the PALSGD update / synchronisation library (CUDA, sm_100a).
 *
 * The library runs the per-step parameter arithmetic of Pseudo-Asynchronous
 * Local SGD (Algorithm 1 of the paper) for K data-parallel workers that live as
 * K replica slots in ONE GPU's memory:
 *
 *   - the inner optimizer step of every worker (AdamW or momentum SGD) with the
 *     rescaled step size alpha_t / (1 - p)                    [Algorithm 1; Eq. (1)]
 *   - the probabilistic pseudo-synchronisation that pulls a worker's local model
 *     x_k toward its copy x of the global model with coefficient
 *     alpha_t * eta_t / p                                     [Algorithm 1; Eq. (2)]
 *   - every H steps the outer synchronisation: average of the K local models
 *     (Sec. 2.2), outer gradient Delta = x - average (Eq. (3)), OuterOPT = SGD
 *     with (Nesterov) momentum (Eq. (4); Sec. 4.3), and the restart of every
 *     worker from the new global model (Sec. 3.1).
 *
 * General rules
 *   - Every entry point returns a palsgd_status (0 = PALSGD_OK, negative = error),
 *     never throws, never exits.  palsgd_strerror() names a status.
 *   - All parameter/gradient/state buffers are DEVICE memory owned by the caller;
 *     they must stay valid until palsgd_destroy().  The library allocates only
 *     its context and a few KB..MB of device tables (chunk table, pointer
 *     tables, a counter block); palsgd_destroy() frees them.
 *   - `stream` arguments are a cudaStream_t passed as void* (NULL = the legacy
 *     default stream).  Work is enqueued asynchronously unless stated otherwise.
 *     Successive calls on one context must be stream-ordered with each other.
 *   - A context is not thread-safe; distinct contexts are independent.
 *   - Buffers need only natural element alignment.  Tensors whose every buffer
 *     is 16-byte aligned take the 128-bit vector path; so do tensors whose
 *     buffers all become 16-byte aligned after the same small number of leading
 *     elements (a packed list at an odd offset), behind a scalar head of those
 *     elements (at most 255: the library prefers the count that puts every
 *     buffer on a multiple of 256 elements' bytes (1024 for fp32, 512 for bf16),
 *     where the kernels run at their full rate; allocate there if you can);
 *     anything else takes a scalar path.  Results are identical.
 *   - Arguments are checked before anything is enqueued: an EINVAL / EALIGN call
 *     has changed nothing.  If a CUDA call fails in the middle of an entry point
 *     (PALSGD_ECUDA), the context is marked failed and every later call that
 *     would read or advance its state returns PALSGD_ESTATE; destroy it.
 *   - Arithmetic: every element operation is one IEEE binary32 operation in the
 *     order documented at each call (no fused multiply-add, round-to-nearest
 *     division and square root).  Scalars (step sizes, bias corrections) are
 *     formed in binary64 and rounded once.
 */
#ifndef PALSGD_H_
#define PALSGD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PALSGD_MAX_WORKERS 64u

typedef struct palsgd_ctx palsgd_ctx;   /* opaque; created by palsgd_init, freed by palsgd_destroy */

typedef enum palsgd_status {
    PALSGD_OK           =  0,
    PALSGD_EINVAL       = -1,   /* NULL pointer, K = 0 or > 64, H = 0, p outside [0,1], bad enum ... */
    PALSGD_EALIGN       = -2,   /* a pointer is not aligned to its element size                      */
    PALSGD_ECUDA        = -3,   /* a CUDA runtime call or a kernel launch failed                     */
    PALSGD_ESTATE       = -4,   /* call not valid in this state (e.g. undefined coefficient)         */
    PALSGD_ENOMEM       = -5,   /* host or device allocation failed                                  */
    PALSGD_EUNSUPPORTED = -6,   /* combination not built                                             */
    /* -7 is not used */
    PALSGD_ETOOBIG      = -8    /* tensor list needs more than the fixed scratch of a no-allocation call */
} palsgd_status;

enum { PALSGD_INNER_ADAMW = 0, PALSGD_INNER_SGDM = 1 };
enum { PALSGD_PREC_FP32 = 0, PALSGD_PREC_BF16_MASTER = 1 };
enum { PALSGD_OUTER_SGD = 0, PALSGD_OUTER_ADAMW = 1 };
enum { PALSGD_SCHED_WARMUP_CONSTANT = 0, PALSGD_SCHED_WARMUP_COSINE = 1 };

/* Algorithm 1's data line: K, p, H, InnerOPT, OuterOPT.  (alpha_t and eta_t are
 * per-call arguments because the paper indexes them by t.) */
typedef struct palsgd_config {
    uint32_t K;               /* number of workers / replica slots, 1..64                        */
    int32_t  inner;           /* PALSGD_INNER_ADAMW | PALSGD_INNER_SGDM                          */
    uint64_t H;               /* outer-sync interval, >= 1                                       */
    double   p;               /* probability of the pseudo-sync branch, in [0, 1]                */
    double   beta1, beta2;    /* AdamW moment decay rates                                        */
    double   eps;             /* AdamW epsilon (added to sqrt of the corrected second moment)    */
    double   weight_decay;    /* AdamW: decoupled; SGD: L2 term added to the gradient            */
    double   momentum;        /* inner SGD momentum (ignored by AdamW)                           */
    double   outer_lr;        /* OuterOPT learning rate                                          */
    double   outer_momentum;  /* OuterOPT momentum; (outer_lr, outer_momentum, nesterov) =       */
    int32_t  outer_nesterov;  /*   (1, 0, 0) is plain averaging (Local SGD / Theorem 1)          */
    int32_t  precision;       /* PALSGD_PREC_FP32 | PALSGD_PREC_BF16_MASTER                      */
    uint64_t seed;            /* seed of the decision stream                                     */
    /* OuterOPT variants of the optimizer ablation (Appendix D).  PALSGD_OUTER_SGD uses
     * outer_lr / outer_momentum / outer_nesterov above; PALSGD_OUTER_ADAMW applies AdamW to
     * the outer gradient with the four constants below and needs palsgd_buffers.outer_v.     */
    int32_t  outer_opt;       /* PALSGD_OUTER_SGD | PALSGD_OUTER_ADAMW                           */
    int32_t  reserved_;       /* set to 0                                                        */
    double   outer_beta1, outer_beta2, outer_eps, outer_weight_decay;
} palsgd_config;

/* Caller-owned device buffers.  Arrays of K*n_tensors pointers are indexed
 * [k * n_tensors + j] (worker k, tensor j); arrays of n_tensors pointers by [j].
 * The pointer ARRAYS themselves are host memory and are copied by palsgd_init. */
typedef struct palsgd_buffers {
    void* const*       param;      /* [K*n] local models x_k: float (FP32) or bfloat16 working
                                      copy (BF16_MASTER; overwritten by init with RNE(master))   */
    const void* const* grad;       /* [K*n] gradients g_k: float (FP32) or bfloat16; read only   */
    float* const*      master;     /* [K*n] fp32 master of x_k (BF16_MASTER) else NULL           */
    float* const*      m;          /* [K*n] AdamW first moment / SGD momentum buffer             */
    float* const*      v;          /* [K*n] AdamW second moment; NULL for SGD                    */
    float* const*      global;     /* [n]   global model copy x (written by init)                */
    float* const*      outer_mom;  /* [n]   OuterOPT momentum buffer u (zeroed by init); first
                                      moment of the outer gradient for PALSGD_OUTER_ADAMW         */
    float* const*      outer_v;    /* [n]   second moment for PALSGD_OUTER_ADAMW (zeroed by init),
                                      else NULL                                                  */
} palsgd_buffers;

/*
 * Create a context (Algorithm 1, initialisation).  Validates everything before
 * touching the GPU.  Then, on `stream`: m, v, outer_mom (and outer_v) <- 0; global[i] <-
 * (x_0[i] + x_1[i] + ... + x_{K-1}[i]) / K, summed in that order (Sec. 2.2; the
 * paper starts all workers from one x^(0), for which this is x^(0)); in
 * BF16_MASTER mode param <- RNE_bf16(master).  Counters t, s_k, n_outer <- 0.
 * numel[j] is the element count of tensor j (0 allowed).  Tensors that are
 * adjacent in memory in every buffer are fused into one segment internally.
 * Errors: EINVAL / EALIGN before any CUDA call; ENOMEM; ECUDA.
 */
int palsgd_init(palsgd_ctx** out, const palsgd_config* cfg, size_t n_tensors,
                const uint64_t* numel, const palsgd_buffers* bufs, void* stream);

/*
 * One pass of Algorithm 1's inner loop body for all K workers, ONE kernel launch (one
 * more, ahead of it, while gradient clipping is on: see palsgd_set_grad_clip).
 * For worker k the kernel draws b_k^(t), Algorithm 1's uniform variate compared with p: the first word r of
 * Philox4x32-10 with key (seed_lo, seed_hi) and counter (t_lo, t_hi, k0 + k, 0), k0 the worker
 * offset (0 unless palsgd_set_worker_offset was called);
 * b = (r < floor(p * 2^32)).  One draw per (worker, step) for the whole model.
 *   b = 1, Eq. (2):  d = x - x_g;  x = x - beta * d,   beta = fl32(alpha_t*eta_t/p).
 *          Gradient, moments and s_k are not touched.
 *   b = 0, Eq. (1):  s_k += 1;  lr = fl32(alpha_t/(1-p)) and
 *     AdamW:  m = b1*m + (1-b1)*g;  v = b2*v + (1-b2)*(g*g);
 *             mh = m / (1-b1^s_k);  vh = v / (1-b2^s_k);
 *             x = x * fl32(1 - lr*wd);  x = x - lr * (mh / (sqrt(vh) + eps))
 *     SGD:    g' = g + wd*x;  m = mu*m + g';  x = x - lr*m
 * In BF16_MASTER mode x above is the fp32 master, g is widened exactly, and the
 * bf16 working copy is rewritten as RNE(master).  Afterwards t += 1 (device side).
 * Does NOT run the outer sync; see palsgd_step.
 * Errors: EINVAL (NULL ctx, non-finite or negative rates); ECUDA.
 */
int palsgd_inner_step(palsgd_ctx* ctx, double lr_t, double eta_t, void* stream);

/*
 * One step of the DDP warm-up phase that precedes Algorithm 1 (Sec. 3.3: training
 * starts with a DDP phase; Sec. 4.1: all Local SGD variants use DDP for the initial
 * steps), ONE kernel launch.  Mini-batch SGD over the K workers:
 *   gbar = (g_0 + g_1 + ... + g_{K-1}) / K          (that order, one division)
 *   one InnerOPT step with the plain step size lr = fl32(alpha_t) -- no 1/(1-p)
 *   rescaling, there is no mixing branch in this phase -- using the formulas of
 *   palsgd_inner_step's b = 0 case with g = gbar.
 * In this phase all workers hold the same model and optimizer state, so the step
 * is taken once, on worker 0's x, m, v and step count, and the result is written
 * to every worker's x, m, v (and bf16 working copy) and to the global model copy
 * x_g; s_k and the bias-correction products of every worker follow worker 0.
 * The outer momentum u is not touched.  No draw; the recorded decisions are 0;
 * t += 1 (the decision stream stays indexed by the global step).  Never runs the
 * outer sync: switch to palsgd_step when the warm-up ends.
 * Errors: EINVAL (NULL ctx, non-finite or negative rate); ECUDA.
 */
int palsgd_ddp_step(palsgd_ctx* ctx, double lr_t, void* stream);

/*
 * A pull imposed on the workers whose bit is set in worker_mask, with the mixing
 * coefficient given directly (the EMA form after Eq. (2): x_k <- (1-beta) x_k +
 * beta x, computed as x - beta*(x - x_g)).  No draw; t, s_k unchanged.
 * Errors: EINVAL (NULL ctx, mask bit >= K, non-finite beta); ECUDA.
 */
int palsgd_pseudo_sync(palsgd_ctx* ctx, uint64_t worker_mask, double beta, void* stream);

/*
 * Outer synchronisation, ONE kernel launch (Algorithm 1, "(t+1) mod H = 0" block):
 *   xbar = (x_0 + x_1 + ... + x_{K-1}) / K      (that order; Sec. 2.2)
 *   Delta = x_g - xbar                          (Eq. (3))
 *   u = mu*u + Delta;  x_g = x_g - lr_out*(Delta + mu*u)   (Nesterov; Eq. (4))
 *                      x_g = x_g - lr_out*u                (outer_nesterov = 0)
 *   x_k = x_g for every k  (Sec. 3.1: every worker restarts from the global model)
 * With PALSGD_OUTER_ADAMW (the ablation's AdamW OuterOPT) the update of x_g is instead, with
 * n = n_outer + 1 and the outer_* constants of the configuration:
 *   u = ob1*u + (1-ob1)*Delta;  v = ob2*v + (1-ob2)*(Delta*Delta);
 *   uh = u / (1-ob1^n);  vh = v / (1-ob2^n);
 *   x_g = x_g * fl32(1 - lr_out*owd);  x_g = x_g - lr_out * (uh / (sqrt(vh) + oeps))
 * lr_out is the configuration's outer_lr or the latest palsgd_set_outer_lr value.
 * Inner optimizer state is kept.  n_outer += 1.  BF16_MASTER: masters are
 * averaged; masters and bf16 working copies are rewritten.
 * Errors: EINVAL (NULL ctx); ECUDA.
 */
int palsgd_outer_sync(palsgd_ctx* ctx, void* stream);

/*
 * The outer synchronisation when the K workers of Algorithm 1 are spread over several GPUs
 * (the deployment the paper itself runs: Algorithm 1's All-Reduce of the outer gradient across
 * workers, an average by Sec. 2.2).  Each GPU holds a context over its K_local workers; the
 * exchange is the caller's collective (e.g. one NCCL all-reduce(sum)), the library supplies the
 * two kernels around it:
 *   1. palsgd_outer_partial:  exchange[i] = x_0[i] + x_1[i] + ... + x_{K_local-1}[i]  (that order)
 *   2. the caller sums the exchange buffers of all GPUs element by element (all-reduce, sum)
 *   3. palsgd_outer_finish:   xbar = exchange[i] / K_total;  then exactly palsgd_outer_sync's
 *      Delta, OuterOPT update of x_g (Eq. (3), Eq. (4)) and the restart of the K_local slots.
 * With one GPU (K_total = K_local, step 2 empty) the result is bit-identical to
 * palsgd_outer_sync.  With G GPUs the sum over k is grouped by GPU, and the order in which step
 * 2 adds the G partial sums is the collective's; the result then differs from the single-GPU one
 * by rounding only (for G = 2 it is one commutative addition, hence unique).  Every GPU must
 * call with the same outer learning rate and K_total; all end with the same x_g and u.
 * The exchange buffer is device memory of palsgd_exchange_numel() floats (the total element
 * count), 16-byte aligned, caller-owned: the tensor list packed back to back, tensor j at the
 * sum of the element counts before it -- the same on every GPU whatever its memory layout.
 * palsgd_outer_finish counts as the outer sync: n_outer += 1.
 * palsgd_set_worker_offset(k0) makes the local workers draw their decisions as workers
 * k0 .. k0+K_local-1 of the job (Algorithm 1's worker index); default 0.
 * Initialisation: palsgd_init sets x_g to the mean of the LOCAL slots.  For the job's global
 * model (the mean over all K_total workers, Sec. 2.2) run, once after palsgd_init on every GPU:
 * palsgd_outer_partial -> the same all-reduce -> palsgd_global_from_exchange, which writes
 * x_g = exchange / K_total and touches nothing else.
 * Errors: EINVAL (NULL, K_total < K_local, k0 + K_local > 2^32); EALIGN; EUNSUPPORTED (an
 * OUTER_SUB_ELEMS value whose stage does not fit in shared memory); ECUDA.
 */
int palsgd_exchange_numel(palsgd_ctx* ctx, uint64_t* n_floats);
int palsgd_set_worker_offset(palsgd_ctx* ctx, uint32_t k0);
int palsgd_outer_partial(palsgd_ctx* ctx, float* exchange, void* stream);
int palsgd_outer_finish(palsgd_ctx* ctx, const float* exchange, uint32_t K_total, void* stream);
int palsgd_global_from_exchange(palsgd_ctx* ctx, const float* exchange, uint32_t K_total, void* stream);

/*
 * The DDP warm-up step (see palsgd_ddp_step; Sec. 3.3, Sec. 4.1) for workers spread over several GPUs,
 * around the same exchange buffer and the caller's all-reduce:
 *   1. palsgd_ddp_partial:  exchange[i] = g_0[i] + ... + g_{K_local-1}[i]   (that order; bf16 widened exactly)
 *   2. all-reduce (sum) of the exchange buffers
 *   3. palsgd_ddp_finish:   gbar = exchange[i] / K_total, then exactly palsgd_ddp_step's optimizer step on
 *      local worker 0's state, written to the K_local slots and to x_g; s_k, t as in palsgd_ddp_step.
 * All ranks hold the same model and state in this phase and receive the same sum, so they stay identical.
 * With one GPU the result is bit-identical to palsgd_ddp_step.  Gradient clipping is not offered in this form
 * (the norm would be that of a gradient living in the exchange buffer).
 * Errors: EINVAL (NULL, K_total < K_local, bad rate); EALIGN; EUNSUPPORTED (clipping on, or DDP_VARIANT 1);
 * ECUDA.
 */
int palsgd_ddp_partial(palsgd_ctx* ctx, float* exchange, void* stream);
int palsgd_ddp_finish(palsgd_ctx* ctx, const float* exchange, uint32_t K_total, double lr_t, void* stream);

/* The outer learning rate of the following outer syncs (it may follow a schedule, e.g. the
 * warm-up + cosine annealing of Appendix B: see palsgd_schedule_value).  Errors: EINVAL. */
int palsgd_set_outer_lr(palsgd_ctx* ctx, double outer_lr);

/*
 * Pure host function: the value at step t of a schedule with a linear warm-up over
 * `warmup` steps from base*start_factor to base, followed by a constant
 * (PALSGD_SCHED_WARMUP_CONSTANT) or by cosine annealing down to min_value at step `total`
 * (PALSGD_SCHED_WARMUP_COSINE; the outer learning-rate schedule of Appendix B):
 *   t <  warmup: base * (start_factor + (1 - start_factor) * t / warmup)
 *   t >= warmup: base, or min_value + (base - min_value) * (1 + cos(pi*tau/(total - warmup))) / 2
 *                with tau = min(t, total) - warmup.
 * Returns NaN for an unknown kind or non-finite arguments.  Feed the result to
 * palsgd_inner_step / palsgd_step (alpha_t, eta_t) or palsgd_set_outer_lr.
 */
double palsgd_schedule_value(int kind, uint64_t t, uint64_t warmup, uint64_t total, double base,
                             double min_value, double start_factor);

/* Algorithm 1, one iteration t: palsgd_inner_step, then palsgd_outer_sync when
 * the number of completed steps is a multiple of H. */
int palsgd_step(palsgd_ctx* ctx, double lr_t, double eta_t, void* stream);

/*
 * One synchronisation cycle of Algorithm 1 -- H iterations of the loop body followed by the
 * outer sync -- as ONE CUDA graph, for models so small that the launches, not the kernels,
 * set the pace.  Possible because the kernels take t, s_k and the bias-correction products
 * from device memory: the H inner launches have identical arguments.
 * palsgd_cycle_capture records the cycle with the given alpha_t, eta_t (constant over the
 * cycle), the current outer learning rate, clip threshold and tuning knobs; it runs nothing
 * and may be called again to replace the recording (e.g. when a schedule moves the rates).
 * It creates a stream and a graph, so call it outside any capture of the caller's own.
 * palsgd_cycle_launch enqueues the recorded cycle on `stream`: t += H, n_outer += 1.
 * Both need t to be a multiple of H (a cycle starts right after a sync, or at t = 0).
 * Results are bit-identical to H calls of palsgd_step.  The gradient buffers are read by each of
 * the H steps as they stand on the device at that moment: work that refills them between steps
 * has to be ordered on the device by the caller (e.g. in a graph of the caller's own, around
 * individual palsgd_inner_step / palsgd_outer_sync launches, which are capturable too).
 * Errors: EINVAL; ESTATE (t not a multiple of H; launch without a recording);
 * EUNSUPPORTED (PALSGD_OUTER_ADAMW, whose scalars change every round; H > 65536); ECUDA.
 */
int palsgd_cycle_capture(palsgd_ctx* ctx, double lr_t, double eta_t);
int palsgd_cycle_launch(palsgd_ctx* ctx, void* stream);

/*
 * palsgd_step with HOST gradients and HOST results (the end-to-end call):
 * copies h_grad[k*n_tensors+j] (host, numel[j] elements of the gradient type;
 * pinned memory makes the copies asynchronous) into the gradient buffers, runs
 * palsgd_step, copies the K decisions of this step to h_decisions (K bytes, may
 * be NULL) and, if this step ended with an outer sync and h_global is not NULL,
 * the new global model to h_global[j] (float, numel[j] each).  *synced (may be
 * NULL) receives 1 if the outer sync ran.  SYNCHRONISES the stream before
 * returning.
 * The gradient of a worker that pulls in this step is not used by Algorithm 1 and is
 * NOT copied (its device buffer keeps what it held); palsgd_decision tells the caller
 * beforehand which workers those are, so it need not produce their gradients at all
 * (their h_grad entries may be NULL).
 * The transfer overlaps the arithmetic: the copies run worker by worker on a stream of
 * the library's own (ordered after the work already enqueued on `stream`), and the part
 * of the inner step that belongs to worker k is launched when its gradient has arrived
 * (K launches per step; with gradient clipping on, or K = 1, one launch after all copies).
 * A worker's SMALL copies (under 2 MB each, both ends 16-byte aligned, at least 8 of them, the
 * sources in pinned memory -- a tensor list held as one allocation per tensor) are performed by
 * one more kernel that reads the host memory directly, instead of one copy-engine transfer each;
 * pageable sources and everything else go through cudaMemcpyAsync.  The data moved is the same.
 * Errors: as palsgd_step; EINVAL for a NULL gradient pointer of a non-empty tensor of a
 * worker that takes a gradient step, and for a NULL entry of h_global (non-empty tensor) on a
 * step that ends with the outer sync -- both found before anything is enqueued.
 */
int palsgd_step_host(palsgd_ctx* ctx, const void* const* h_grad, double lr_t, double eta_t,
                     float* const* h_global, uint8_t* h_decisions, int* synced, void* stream);

/*
 * Read the counters (SYNCHRONISES the stream): t = completed steps, s_k[K] =
 * gradient steps taken by worker k, n_outer = outer syncs, last_b[K] = decisions
 * of the latest inner step.  Any output pointer may be NULL.
 * Errors: ESTATE if the device-side t disagrees with the host mirror; ECUDA.
 */
int palsgd_get_counters(palsgd_ctx* ctx, uint64_t* t, uint64_t* s_k, uint64_t* n_outer,
                        uint8_t* last_b, void* stream);

/* Resume: set t, s_k[K], n_outer (the decision stream is a pure function of
 * (seed, t, k), so a restored run continues bit-exactly).  Enqueued on stream. */
int palsgd_set_counters(palsgd_ctx* ctx, uint64_t t, const uint64_t* s_k, uint64_t n_outer,
                        void* stream);

/*
 * Global-norm gradient clipping (Appendix B: the GPT-Neo runs clip their gradients; no
 * threshold is given, so it is a parameter here).  max_norm > 0 turns it
 * on for the following palsgd_inner_step / palsgd_step / palsgd_ddp_step calls,
 * 0 turns it off (the default).  Convention of the software the paper ran
 * (clip_grad_norm_), per worker k that takes a gradient step:
 *   sumsq_k = the exact sum over the worker's WHOLE gradient (all tensors) of g^2,
 *             rounded once to binary64
 *   c_k = fl32(min(1, max_norm / (sqrt(sumsq_k) + 1e-6)))     (binary64, rounded once)
 *   g <- g * c_k (one binary32 multiplication) before InnerOPT sees it.
 * Workers that pull in a step have no norm taken.  In the DDP phase the one norm is
 * that of the averaged gradient gbar.  Costs one extra kernel launch per step that
 * reads every gradient once more.
 * Errors: EINVAL (NULL ctx, negative or non-finite max_norm).
 */
int palsgd_set_grad_clip(palsgd_ctx* ctx, double max_norm);

/* The sums of squares and clip coefficients of the latest clipped step (K each; either
 * pointer may be NULL; entries of workers that pulled keep their previous values;
 * before the first clipped step: 0 and 1).  SYNCHRONISES the stream. */
int palsgd_get_grad_norms(palsgd_ctx* ctx, double* sumsq, float* clip, void* stream);

/* Number of kernels this context has launched so far (host-side count). */
int palsgd_get_launch_count(palsgd_ctx* ctx, uint64_t* n_launches);

/* What palsgd_init made of the tensor list (the multi-tensor launch metadata): the number of
 * segments (maximal runs of tensors that are adjacent in memory in every buffer), of chunk-table
 * entries (pieces of a segment of at most *chunk_elems elements; one work item of the inner kernel
 * per worker each) and the chunk size.  Any output pointer may be NULL.  Errors: EINVAL. */
int palsgd_get_layout(palsgd_ctx* ctx, uint64_t* n_segments, uint64_t* n_chunks, uint32_t* chunk_elems);

/* The same report WITHOUT a context and without touching the GPU: what palsgd_init would make of this
 * tensor list (the multi-tensor launch metadata of the path).  A pure host function of the configuration,
 * the sizes and the ADDRESSES in `bufs` (same tables as for palsgd_init; nothing they point to is read,
 * so it may be called before the buffers hold anything, or from a process without a GPU).
 * Per segment i < *n_segments, if the array pointers are non-NULL (capacity: n_tensors entries each):
 *   seg_first_tensor[i], seg_n_tensors[i]  the run of tensors fused into it (tensors adjacent in every buffer;
 *                                          empty tensors inside a run are skipped over, an all-empty run is dropped)
 *   seg_head[i]   leading elements handled by the scalar path so that the rest is aligned in every buffer
 *                 (see the alignment rule above): 0..255, or -1 = the whole segment takes the scalar path
 * Errors: exactly palsgd_init's argument errors (EINVAL, EALIGN); no other. */
int palsgd_plan_layout(const palsgd_config* cfg, size_t n_tensors, const uint64_t* numel,
                       const palsgd_buffers* bufs, uint64_t* n_segments, uint64_t* n_chunks,
                       uint32_t* chunk_elems, uint64_t* seg_first_tensor, uint64_t* seg_n_tensors,
                       int32_t* seg_head);

/* Launch-shape knobs (advanced; results never depend on them).  Setting any of them drops a cycle recorded by
 * palsgd_cycle_capture (palsgd_cycle_launch then returns ESTATE until the cycle is captured again).
 * *_GRID_CAP: the largest grid a launch may use, CTAs looping over work items
 * beyond it; 0 (default) = one CTA per work item.
 * INNER_VARIANT: 0 = the fused inner kernel as a persistent grid that draws its work items from a
 * queue in device memory (default); 18 = the same kernel with one CTA per work item.
 * OUTER_SUB_ELEMS: elements per work item of the outer kernel, a multiple of 1024; default 1024
 * (4096 for K = 5..7, 2048 for K <= 2).  DDP_SUB_ELEMS: the same for the DDP warm-up kernel (default 1024).  Setting either rebuilds
 * a device table: the call synchronises the device and must not be made during stream capture.
 * DDP_VARIANT: how the DDP warm-up kernel writes its result to the K slots: 1 = 128-bit stores
 * by every thread, 2 = staged in shared memory and fanned out by bulk asynchronous stores;
 * 0 = the library's default (2).
 * OUTER_VARIANT: the same choice for the outer-sync kernel.
 * OUTER_DYNAMIC: outer-sync and DDP kernels as a persistent grid of that many CTAs per SM that
 * draws its work items from a queue; 0 = one CTA per work item.  Until this knob is set the
 * library uses its defaults. */
enum { PALSGD_TUNE_INNER_GRID_CAP = 0, PALSGD_TUNE_OUTER_GRID_CAP = 1, PALSGD_TUNE_INNER_VARIANT = 2,
       PALSGD_TUNE_OUTER_SUB_ELEMS = 5, PALSGD_TUNE_DDP_SUB_ELEMS = 6, PALSGD_TUNE_DDP_VARIANT = 7,
       PALSGD_TUNE_OUTER_VARIANT = 8, PALSGD_TUNE_OUTER_DYNAMIC = 9 };
int palsgd_set_tuning(palsgd_ctx* ctx, int knob, int64_t value);

/* The branch draw as a pure host function: 1 = pseudo-sync, 0 = gradient step;
 * negative status on bad arguments (p outside [0,1]).  k is the worker's index in the job. */
int palsgd_decision(uint64_t seed, uint64_t t, uint32_t k, double p);

/* Text for a status; the CUDA error string of the latest ECUDA on ctx (or ""). */
const char* palsgd_strerror(int status);
const char* palsgd_last_cuda_error(palsgd_ctx* ctx);

/*
 * Outer synchronisation WITHOUT any allocation (the paper has no counterpart:
 * this entry point exists for the way the library gets embedded, not for the
 * method).  Same arithmetic, same kernel and same results as palsgd_outer_sync,
 * for callers that are not allowed to allocate device memory at the point where
 * they synchronise: code running inside a framework whose caching allocator
 * owns all of the GPU's memory, inside a region where cudaMalloc's implicit
 * device-wide synchronisation is unacceptable, or in a process whose memory
 * budget is fixed up front.  Such callers cannot use palsgd_init, which
 * allocates the launch tables.  Here the tables live in a fixed array of
 * PALSGD_NOALLOC_SCRATCH_BYTES that is part of the library image: every GPU
 * that loads the library holds that much memory until the process exits.
 *
 * No context: the caller passes the buffers on every call.  Layout as in
 * palsgd_buffers: param/master are [K*n_tensors] device pointers indexed
 * [k*n_tensors + j], global/outer_mom are [n_tensors]; the pointer ARRAYS are
 * host memory.  FP32: param = float local models, master = NULL.  BF16_MASTER:
 * master = fp32 local models (averaged and rewritten), param = bf16 working
 * copies (rewritten as RNE of the new global model).  numel[j] = 0 is allowed.
 * The call rebuilds the tables, copies them into the array on `stream`, and
 * launches one kernel on `stream`.  It calls neither cudaMalloc nor cudaFree nor
 * any other allocating routine, on the device or on the host.  The tables come
 * from ordinary (pageable) host memory inside the library, so the copy makes
 * the HOST wait until the work enqueued on `stream` before this call has
 * finished; the kernel itself then runs asynchronously, and work on other
 * streams is not affected.
 *
 * Limit: the tables need 16 bytes per started block of 8192 elements of every
 * tensor, plus 8 bytes per (worker, non-empty tensor) pointer (twice that in
 * BF16_MASTER mode) and 16 bytes per non-empty tensor, each table rounded up to
 * 256 bytes.  If that exceeds PALSGD_NOALLOC_SCRATCH_BYTES the call returns
 * PALSGD_ETOOBIG and does nothing (1 MiB covers about 5*10^8 parameters in a
 * few hundred tensors at K = 8).
 *
 * Sharing: all calls on a device use the one array, and it keeps the previous
 * call's tables.  Each call overwrites everything it will read, so nothing has
 * to be cleared; but two calls whose GPU work can overlap (different streams
 * without an ordering between them, or several host threads on different
 * streams) race on the array and give undefined results.  Order them on one
 * stream, or with events.  Host threads are serialised inside the call.
 *
 * First call on each device: looks up the array's device address (a runtime
 * call that is made once per device and cached, with that device current).
 *
 * Never under stream capture, first call or later: the table copy would be
 * recorded as a node that re-reads the library's host buffer, and the kernel
 * node would keep this call's table sizes, at every replay, after later calls
 * have put other tables there.  A call on a capturing stream returns
 * PALSGD_ESTATE and enqueues nothing.
 * Errors: EINVAL, EALIGN, ETOOBIG before any CUDA call; ESTATE (capturing
 * stream); ECUDA.
 */
#define PALSGD_NOALLOC_SCRATCH_BYTES (1u << 20)
int palsgd_outer_sync_noalloc(uint32_t K, int32_t precision, size_t n_tensors,
                              const uint64_t* numel, void* const* param, float* const* master,
                              float* const* global, float* const* outer_mom, double outer_lr,
                              double outer_momentum, int32_t outer_nesterov, void* stream);

/* Free the context and its device tables.  NULL is accepted.  The caller's
 * buffers are not touched. */
void palsgd_destroy(palsgd_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* PALSGD_H_ */
