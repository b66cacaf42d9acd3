/*
 * PALSGD oracle -- Algorithm 1, executed step by step.   TEST INFRASTRUCTURE ONLY.
 *
 * Compiled twice: -DREAL=float -DSUFFIX=f32 (the parity reference: every
 * element operation is one IEEE binary32 operation, no fused multiply-add) and
 * -DREAL=double -DSUFFIX=f64 (an accuracy yard-stick).  Build flags must
 * include -ffp-contract=off.
 *
 * Notation follows the paper: K workers, x_k local model, x the global model
 * copy (x_g here), alpha_t inner learning rate, eta_t mixing rate, p mixing
 * probability, H sync interval.  u is the outer (Nesterov) momentum buffer,
 * s_k the number of gradient steps worker k has taken.
 *
 *   Algorithm 1, branch draw            -> draw in FN(inner_step)
 *   Algorithm 1 / Eq. (2), pseudo-sync  -> pull_worker
 *   Algorithm 1 / Eq. (1), gradient step-> adamw_worker / sgdm_worker with
 *                                          step size alpha_t / (1 - p)
 *   Sec. 2.2 average, Eq. (3), Eq. (4)  -> FN(outer_sync)
 *   Sec. 3.3 / Sec. 4.1 DDP warm-up     -> FN(ddp_step)
 *
 * The paper names its optimizers without printing them (Sec. 4.3): InnerOPT is
 * AdamW (decoupled weight decay, bias-corrected) or momentum SGD, OuterOPT is
 * SGD with Nesterov momentum.  Their textbook forms are written out below and
 * pinned against torch.optim on the CPU by the tests.
 *
 * The model is one flat vector of P elements: with uniform hyper-parameters a
 * tensor list is its concatenation, because every operation is elementwise.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>

#ifndef REAL
#error "compile with -DREAL=float|double -DSUFFIX=f32|f64"
#endif
#define CAT2(a, b) a##_##b
#define CAT(a, b) CAT2(a, b)
#define FN(name) CAT(CAT(palsgd_oracle, name), SUFFIX)

int      palsgd_oracle_decision(uint64_t seed, uint64_t t, uint32_t k, double p);
float    palsgd_oracle_bf16_to_f32(uint16_t h);
uint16_t palsgd_oracle_bf16_from_f32(float f);
uint16_t palsgd_oracle_bf16_from_f64(double d);
double   palsgd_oracle_sumsq_f32(const float *g, uint64_t n);
double   palsgd_oracle_sumsq_f64(const double *g, uint64_t n);
double   palsgd_oracle_sumsq_bf16(const uint16_t *g, uint64_t n);
double   palsgd_oracle_clip_coef(double sumsq, double max_norm);

typedef struct {
    /* Algorithm 1's data line */
    uint32_t K;              /* number of workers                                  */
    uint64_t H;              /* sync interval                                      */
    double   p;              /* probability of the mixing (pseudo-sync) step       */
    int32_t  inner;          /* InnerOPT: 0 AdamW, 1 momentum SGD                  */
    double   beta1, beta2, eps, weight_decay;   /* AdamW constants / weight decay  */
    double   momentum;       /* inner SGD momentum                                 */
    double   outer_lr, outer_momentum;          /* OuterOPT                        */
    int32_t  outer_nesterov; /* 1: Nesterov; 0: plain momentum                     */
    uint64_t seed;           /* decision stream seed                               */
    int32_t  precision;      /* 0: fp32 params; 1: bf16 working copy + master      */
    uint64_t P;              /* model size                                         */
    /* state, arrays owned by the caller */
    REAL     *x;             /* [K][P] local models x_k (the master in mode 1)     */
    REAL     *m, *v;         /* [K][P] AdamW moments; SGD uses m as its buffer     */
    REAL     *xg;            /* [P] global model copy x                            */
    REAL     *u;             /* [P] outer momentum                                 */
    uint16_t *xw;            /* [K][P] bf16 working params (mode 1) or NULL        */
    uint64_t  t;             /* completed steps                                    */
    uint64_t *s;             /* [K] gradient steps taken by worker k               */
    uint64_t  n_outer;       /* outer syncs performed                              */
    double   *pow1, *pow2;   /* [K] beta1^s_k, beta2^s_k (running products)        */
    uint8_t  *last_b;        /* [K] decisions of the latest step                   */
    /* global-norm gradient clipping (Appendix B: the GPT-Neo runs clip their gradients) */
    double    max_grad_norm; /* threshold; 0 = no clipping                         */
    const double *forced_sumsq; /* NULL, or [K] sums of squares to use instead of
                                computing them (sampled replays of a large run)   */
    double   *sumsq;         /* [K] sum of squares of the latest gradients seen    */
    double   *clipc;         /* [K] coefficient the latest gradient was scaled by  */
    /* OuterOPT variants of the optimizer ablation (Appendix D): 0 = SGD with
     * (Nesterov) momentum as above, 1 = AdamW applied to the outer gradient    */
    int32_t   outer_opt;
    double    outer_beta1, outer_beta2, outer_eps, outer_weight_decay;
    REAL     *uv;            /* [P] second outer moment (outer_opt = 1) or NULL    */
    double    opow1, opow2;  /* outer_beta1^n_outer, outer_beta2^n_outer           */
    /* Workers spread over G machines (the paper's own deployment: Algorithm 1's All-Reduce across
     * workers; Sec. 2.2: an average).  The sum over the K workers is then formed in two levels: each
     * machine adds up its own K/G consecutive workers in ascending order, and the G partial sums are
     * added in ascending order of the machines.  0 or 1 = one level, ascending k (K workers on one GPU). */
    uint32_t  sum_groups;
} FN(state);

static uint16_t to_bf16(REAL a)
{
    return sizeof(REAL) == 4 ? palsgd_oracle_bf16_from_f32((float)a)
                             : palsgd_oracle_bf16_from_f64((double)a);
}

/* Working copy follows the master after every write of the master (mode 1). */
static void refresh_working(FN(state) *st, uint32_t k)
{
    if (st->precision != 1) return;
    REAL *x = st->x + (size_t)k * st->P;
    uint16_t *xw = st->xw + (size_t)k * st->P;
    #pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)st->P; ++i) xw[i] = to_bf16(x[i]);
}

/* Sum of the K local models at element i: ascending k, or (sum_groups > 1) per machine first and
 * then across the machines, both ascending. */
static REAL sum_over_workers(const FN(state) *st, size_t i)
{
    const uint32_t K = st->K;
    const size_t P = st->P;
    REAL sum = st->x[i];
    if (st->sum_groups > 1) {
        const uint32_t per = K / st->sum_groups;
        for (uint32_t gi = 0; gi < st->sum_groups; ++gi) {
            REAL part = st->x[(size_t)(gi * per) * P + i];
            for (uint32_t k = gi * per + 1; k < (gi + 1) * per; ++k) part = part + st->x[(size_t)k * P + i];
            sum = gi == 0 ? part : sum + part;
        }
    } else {
        for (uint32_t k = 1; k < K; ++k) sum = sum + st->x[(size_t)k * P + i];
    }
    return sum;
}

/* Set-up: x_g = (1/K) sum_k x_k (Sec. 2.2 average; Algorithm 1 starts every
 * worker from the same x^(0), for which this is x^(0) up to the rounding of the
 * sum and the division), all optimizer state zero, counters zero. */
void FN(init)(FN(state) *st)
{
    const uint32_t K = st->K;
    const size_t P = st->P;
    #pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)P; ++i) {
        st->xg[i] = sum_over_workers(st, (size_t)i) / (REAL)K;
        st->u[i] = (REAL)0;
    }
    for (uint32_t k = 0; k < K; ++k) {
        #pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < (int64_t)P; ++i) {
            st->m[(size_t)k * P + i] = (REAL)0;
            if (st->v) st->v[(size_t)k * P + i] = (REAL)0;
        }
        st->s[k] = 0; st->pow1[k] = 1.0; st->pow2[k] = 1.0; st->last_b[k] = 0;
        refresh_working(st, k);
    }
    st->t = 0; st->n_outer = 0;
    st->opow1 = 1.0; st->opow2 = 1.0;
    if (st->uv) {
        #pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < (int64_t)P; ++i) st->uv[i] = (REAL)0;
    }
}

/* Eq. (2): x_k <- x_k - beta (x_k - x), beta = alpha_t eta_t / p.
 * Touches nothing but x_k: no gradient, no optimizer state, no step count. */
static void pull_worker(FN(state) *st, uint32_t k, REAL beta)
{
    REAL *x = st->x + (size_t)k * st->P;
    const REAL *xg = st->xg;
    #pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)st->P; ++i) {
        REAL d = x[i] - xg[i];
        x[i] = x[i] - beta * d;
    }
    refresh_working(st, k);
}

/* InnerOPT = AdamW with step size lr (Eq. (1): lr = alpha_t / (1 - p)). */
static void adamw_worker(FN(state) *st, uint32_t k, const float *g32, const uint16_t *g16,
                         double lr_d, REAL clip)
{
    const size_t P = st->P;
    REAL *x = st->x + (size_t)k * P, *m = st->m + (size_t)k * P, *v = st->v + (size_t)k * P;
    st->s[k] += 1;
    st->pow1[k] *= st->beta1;
    st->pow2[k] *= st->beta2;
    const REAL lr    = (REAL)lr_d;
    const REAL b1    = (REAL)st->beta1,         b2    = (REAL)st->beta2;
    const REAL omb1  = (REAL)(1.0 - st->beta1), omb2  = (REAL)(1.0 - st->beta2);
    const REAL bc1   = (REAL)(1.0 - st->pow1[k]);      /* 1 - beta1^s_k */
    const REAL bc2   = (REAL)(1.0 - st->pow2[k]);      /* 1 - beta2^s_k */
    const REAL decay = (REAL)(1.0 - lr_d * st->weight_decay);
    const REAL eps   = (REAL)st->eps;
    #pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)P; ++i) {
        REAL g = g32 ? (REAL)g32[i] : (REAL)palsgd_oracle_bf16_to_f32(g16[i]);
        g = g * clip;                                   /* clipped gradient (clip = 1: unchanged) */
        REAL mi = b1 * m[i] + omb1 * g;
        REAL vi = b2 * v[i] + omb2 * (g * g);
        REAL mhat = mi / bc1;
        REAL vhat = vi / bc2;
        REAL xi = x[i] * decay;                         /* decoupled weight decay */
        REAL root = sizeof(REAL) == 4 ? (REAL)sqrtf((float)vhat) : (REAL)sqrt((double)vhat);
        xi = xi - lr * (mhat / (root + eps));
        m[i] = mi; v[i] = vi; x[i] = xi;
    }
    refresh_working(st, k);
}

/* InnerOPT = momentum SGD with step size lr; L2 decay added to the gradient,
 * buffer starts at zero, no dampening, no Nesterov. */
static void sgdm_worker(FN(state) *st, uint32_t k, const float *g32, const uint16_t *g16,
                        double lr_d, REAL clip)
{
    const size_t P = st->P;
    REAL *x = st->x + (size_t)k * P, *buf = st->m + (size_t)k * P;
    st->s[k] += 1;
    const REAL lr = (REAL)lr_d, mu = (REAL)st->momentum, wd = (REAL)st->weight_decay;
    #pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)P; ++i) {
        REAL g = g32 ? (REAL)g32[i] : (REAL)palsgd_oracle_bf16_to_f32(g16[i]);
        g = g * clip;
        REAL gp = g + wd * x[i];
        REAL b = mu * buf[i] + gp;
        buf[i] = b;
        x[i] = x[i] - lr * b;
    }
    refresh_working(st, k);
}

/* One pass of Algorithm 1's inner loop body for all K workers (without the
 * synchronisation test).  grads: [K][P], float32 (mode 0) or bf16 bits (mode 1).
 * forced_b: NULL to draw the decisions, or K bytes (0/1) to impose them (used
 * by hand traces only).  Returns 0, or -1 when a needed coefficient is
 * undefined (a pull with p = 0, a gradient step with p = 1). */
int FN(inner_step)(FN(state) *st, const void *grads, double alpha_t, double eta_t,
                   const uint8_t *forced_b)
{
    /* refuse, before touching anything, a step whose coefficient is undefined */
    for (uint32_t k = 0; k < st->K; ++k) {
        int b = forced_b ? (forced_b[k] != 0)
                         : palsgd_oracle_decision(st->seed, st->t, k, st->p);
        if (b ? !(st->p > 0.0) : !(st->p < 1.0)) return -1;
    }
    for (uint32_t k = 0; k < st->K; ++k) {
        /* b ~ U[0,1]; if b <= p */
        int b = forced_b ? (forced_b[k] != 0)
                         : palsgd_oracle_decision(st->seed, st->t, k, st->p);
        st->last_b[k] = (uint8_t)b;
        if (b) {
            /* pseudo-synchronization step */
            REAL beta = (REAL)(alpha_t * eta_t / st->p);
            pull_worker(st, k, beta);
        } else {
            /* gradient step: InnerOPT(x_k, g_k, alpha_t / (1 - p)) */
            double lr_d = alpha_t / (1.0 - st->p);
            const float *g32 = st->precision == 0 ? (const float *)grads + (size_t)k * st->P : NULL;
            const uint16_t *g16 = st->precision == 1 ? (const uint16_t *)grads + (size_t)k * st->P : NULL;
            /* clip this worker's gradient to global norm max_grad_norm before InnerOPT sees it */
            REAL clip = (REAL)1;
            if (st->max_grad_norm > 0.0) {
                double ss = st->forced_sumsq ? st->forced_sumsq[k]
                          : g32 ? palsgd_oracle_sumsq_f32(g32, st->P) : palsgd_oracle_sumsq_bf16(g16, st->P);
                double c = palsgd_oracle_clip_coef(ss, st->max_grad_norm);
                st->sumsq[k] = ss; st->clipc[k] = c;
                clip = (REAL)c;
            }
            if (st->inner == 0) adamw_worker(st, k, g32, g16, lr_d, clip);
            else                sgdm_worker(st, k, g32, g16, lr_d, clip);
        }
    }
    st->t += 1;
    return 0;
}

/* A pull imposed on the workers whose bit is set in worker_mask, with the
 * mixing coefficient given directly (EMA form of Eq. (2)); no draw, no
 * counter changes. */
void FN(pseudo_sync)(FN(state) *st, uint64_t worker_mask, double beta)
{
    for (uint32_t k = 0; k < st->K; ++k)
        if ((worker_mask >> k) & 1u) pull_worker(st, k, (REAL)beta);
}

/* Outer synchronisation: average of the local models (Sec. 2.2), outer
 * gradient Delta = x - average (Eq. (3)), OuterOPT = SGD with (Nesterov)
 * momentum (Eq. (4)), then every worker restarts from the new global model.
 * The inner optimizer state is left as it is. */
void FN(outer_sync)(FN(state) *st)
{
    const uint32_t K = st->K;
    const size_t P = st->P;
    const REAL mu = (REAL)st->outer_momentum, lr = (REAL)st->outer_lr;
    /* OuterOPT = AdamW on the outer gradient Delta (one of the ablation's choices): the textbook
     * form used for InnerOPT, with u as first and uv as second moment and n_outer + 1 as step count */
    if (st->outer_opt == 1) {
        st->opow1 *= st->outer_beta1;
        st->opow2 *= st->outer_beta2;
    }
    const REAL ob1 = (REAL)st->outer_beta1, ob2 = (REAL)st->outer_beta2;
    const REAL oomb1 = (REAL)(1.0 - st->outer_beta1), oomb2 = (REAL)(1.0 - st->outer_beta2);
    const REAL obc1 = (REAL)(1.0 - st->opow1), obc2 = (REAL)(1.0 - st->opow2);
    const REAL odecay = (REAL)(1.0 - st->outer_lr * st->outer_weight_decay);
    const REAL oeps = (REAL)st->outer_eps;
    #pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)P; ++i) {
        REAL sum = sum_over_workers(st, (size_t)i);
        REAL xbar  = sum / (REAL)K;
        REAL delta = st->xg[i] - xbar;
        if (st->outer_opt == 1) {
            REAL mi = ob1 * st->u[i] + oomb1 * delta;
            REAL vi = ob2 * st->uv[i] + oomb2 * (delta * delta);
            REAL mhat = mi / obc1;
            REAL vhat = vi / obc2;
            REAL xi = st->xg[i] * odecay;
            REAL root = sizeof(REAL) == 4 ? (REAL)sqrtf((float)vhat) : (REAL)sqrt((double)vhat);
            xi = xi - lr * (mhat / (root + oeps));
            st->u[i] = mi; st->uv[i] = vi; st->xg[i] = xi;
            for (uint32_t k = 0; k < K; ++k) st->x[(size_t)k * P + i] = xi;
            continue;
        }
        REAL ui    = mu * st->u[i] + delta;
        REAL step  = st->outer_nesterov ? (delta + mu * ui) : ui;
        REAL xnew  = st->xg[i] - lr * step;
        st->u[i]  = ui;
        st->xg[i] = xnew;
        for (uint32_t k = 0; k < K; ++k) st->x[(size_t)k * P + i] = xnew;
    }
    for (uint32_t k = 0; k < K; ++k) refresh_working(st, k);
    st->n_outer += 1;
}

/* DDP warm-up step (Sec. 3.3: training begins with a DDP phase; Sec. 4.1: Local SGD,
 * DiLoCo and PALSGD all use DDP during the initial steps).
 * Mini-batch SGD over K workers: the gradients are averaged,
 *     gbar = (g_0 + g_1 + ... + g_{K-1}) / K      (ascending k, one division),
 * and every worker applies the same InnerOPT step with the plain step size
 * alpha_t (no 1/(1-p) rescaling: there is no mixing branch in this phase).
 * In this phase all workers hold the same model and the same optimizer state;
 * the step is therefore taken once, on worker 0's model and state, and the
 * result is written to every worker, and to the global model copy x, which in
 * this phase is that common model.  s_k and the bias-correction products of
 * every worker follow worker 0.  No draw is made; the decisions of the step are
 * recorded as 0; t advances; no outer synchronisation happens in this phase.
 * grads: [K][P], float32 (mode 0) or bf16 bits (mode 1). */
void FN(ddp_step)(FN(state) *st, const void *grads, double alpha_t)
{
    const uint32_t K = st->K;
    const size_t P = st->P;
    const float *g32 = st->precision == 0 ? (const float *)grads : NULL;
    const uint16_t *g16 = st->precision == 1 ? (const uint16_t *)grads : NULL;
    REAL *x = st->x, *m = st->m, *v = st->v;          /* worker 0 */

    st->s[0] += 1;
    if (st->inner == 0) { st->pow1[0] *= st->beta1; st->pow2[0] *= st->beta2; }
    const REAL lr    = (REAL)alpha_t;
    const REAL b1    = (REAL)st->beta1,         b2    = (REAL)st->beta2;
    const REAL omb1  = (REAL)(1.0 - st->beta1), omb2  = (REAL)(1.0 - st->beta2);
    const REAL bc1   = (REAL)(1.0 - st->pow1[0]);
    const REAL bc2   = (REAL)(1.0 - st->pow2[0]);
    const REAL decay = (REAL)(1.0 - alpha_t * st->weight_decay);
    const REAL eps   = (REAL)st->eps;
    const REAL mu    = (REAL)st->momentum, wd = (REAL)st->weight_decay;

    /* averaged gradient */
    REAL *gbar = (REAL *)malloc((P ? P : 1) * sizeof(REAL));
    if (!gbar) return;
    #pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)P; ++i) {
        /* ascending k; with the workers on several machines (sum_groups > 1) per machine first, then
         * across the machines -- the order in which a DDP all-reduce of per-machine sums adds them */
        #define GRAD_AT(k) (g32 ? (REAL)g32[(size_t)(k) * P + i] : (REAL)palsgd_oracle_bf16_to_f32(g16[(size_t)(k) * P + i]))
        REAL sum = GRAD_AT(0);
        if (st->sum_groups > 1) {
            const uint32_t per = K / st->sum_groups;
            for (uint32_t gi = 0; gi < st->sum_groups; ++gi) {
                REAL part = GRAD_AT(gi * per);
                for (uint32_t k = gi * per + 1; k < (gi + 1) * per; ++k) part = part + GRAD_AT(k);
                sum = gi == 0 ? part : sum + part;
            }
        } else {
            for (uint32_t k = 1; k < K; ++k) sum = sum + GRAD_AT(k);
        }
        #undef GRAD_AT
        gbar[i] = sum / (REAL)K;
    }
    /* in this phase the clip applies to the averaged gradient */
    REAL clip = (REAL)1;
    if (st->max_grad_norm > 0.0) {
        double ssq = st->forced_sumsq ? st->forced_sumsq[0]
                   : sizeof(REAL) == 4 ? palsgd_oracle_sumsq_f32((const float *)(const void *)gbar, P)
                                       : palsgd_oracle_sumsq_f64((const double *)(const void *)gbar, P);
        double c = palsgd_oracle_clip_coef(ssq, st->max_grad_norm);
        for (uint32_t k = 0; k < K; ++k) { st->sumsq[k] = ssq; st->clipc[k] = c; }
        clip = (REAL)c;
    }

    #pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)P; ++i) {
        REAL g = gbar[i] * clip;
        REAL xi;
        if (st->inner == 0) {
            REAL mi = b1 * m[i] + omb1 * g;
            REAL vi = b2 * v[i] + omb2 * (g * g);
            REAL mhat = mi / bc1;
            REAL vhat = vi / bc2;
            xi = x[i] * decay;
            REAL root = sizeof(REAL) == 4 ? (REAL)sqrtf((float)vhat) : (REAL)sqrt((double)vhat);
            xi = xi - lr * (mhat / (root + eps));
            for (uint32_t k = 0; k < K; ++k) { m[(size_t)k * P + i] = mi; v[(size_t)k * P + i] = vi; }
        } else {
            REAL gp = g + wd * x[i];
            REAL b = mu * m[i] + gp;
            xi = x[i] - lr * b;
            for (uint32_t k = 0; k < K; ++k) m[(size_t)k * P + i] = b;
        }
        for (uint32_t k = 0; k < K; ++k) x[(size_t)k * P + i] = xi;
        st->xg[i] = xi;
    }
    free(gbar);
    for (uint32_t k = 0; k < K; ++k) {
        st->s[k] = st->s[0]; st->pow1[k] = st->pow1[0]; st->pow2[k] = st->pow2[0];
        st->last_b[k] = 0;
        refresh_working(st, k);
    }
    st->t += 1;
}

/* Algorithm 1, one iteration t: inner loop body, then "if (t+1) mod H = 0". */
int FN(step)(FN(state) *st, const void *grads, double alpha_t, double eta_t,
             const uint8_t *forced_b)
{
    int rc = FN(inner_step)(st, grads, alpha_t, eta_t, forced_b);
    if (rc) return rc;
    if (st->t % st->H == 0) FN(outer_sync)(st);
    return 0;
}
