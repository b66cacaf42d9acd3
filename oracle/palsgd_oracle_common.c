/*
 * PALSGD oracle -- shared integer pieces.   TEST INFRASTRUCTURE ONLY.
 *
 * This directory is the slow, plain CPU statement of what the CUDA library
 * must compute.  It is used by the tests, by the smoke check and by the
 * benchmark's CPU-baseline leg; the product path never calls it, and it shares
 * no code with the CUDA sources.
 *
 * Contents of this file:
 *   - Philox4x32-10, written from its published definition (Salmon, Moraes,
 *     Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC'11);
 *   - the Bernoulli branch draw of Algorithm 1 ("b ~ U[0,1]; if b <= p"),
 *     realised on a 32-bit grid;
 *   - round-to-nearest-even conversion to bfloat16 (top 16 bits of binary32).
 *
 * Pins (tests/test_oracle_philox.py, tests/test_oracle_bf16.py): the Philox
 * words are compared with cuRAND's host-side PHILOX4_32_10 generator through
 * its public API; decision frequencies are checked against p; the bf16
 * rounding is checked exhaustively against exact rational arithmetic.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
static int oracle_thread_id(void)    { return omp_get_thread_num(); }
static int oracle_thread_count(void) { return omp_get_num_threads(); }
#else
static int oracle_thread_id(void)    { return 0; }
static int oracle_thread_count(void) { return 1; }
#endif

/* ---- Philox4x32-10 ------------------------------------------------------ */

static void mulhilo32(uint32_t a, uint32_t b, uint32_t *hi, uint32_t *lo)
{
    uint64_t prod = (uint64_t)a * (uint64_t)b;
    *hi = (uint32_t)(prod >> 32);
    *lo = (uint32_t)prod;
}

void palsgd_oracle_philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2],
                                 uint32_t out[4])
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;   /* round multipliers   */
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;   /* Weyl key increments */
    uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
    uint32_t k0 = key_in[0], k1 = key_in[1];
    for (int round = 0; round < 10; ++round) {
        uint32_t hi0, lo0, hi1, lo1;
        if (round > 0) { k0 += W0; k1 += W1; }
        mulhilo32(M0, c0, &hi0, &lo0);
        mulhilo32(M1, c2, &hi1, &lo1);
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* ---- Branch draw (Algorithm 1: "b ~ U[0,1]; if b <= p") ------------------ */

/* The uniform draw is the first Philox word r in [0, 2^32); the test "b <= p"
 * becomes r < floor(p * 2^32).  p = 0 never pulls, p = 1 always pulls.        */
uint64_t palsgd_oracle_threshold(double p)
{
    return (uint64_t)floor(p * 4294967296.0);
}

/* One draw per (worker k, step t), the same for the worker's whole model.
 * counter = (t_lo, t_hi, k, 0), key = (seed_lo, seed_hi), word 0 is used.    */
uint32_t palsgd_oracle_draw_word(uint64_t seed, uint64_t t, uint32_t k)
{
    uint32_t ctr[4] = { (uint32_t)t, (uint32_t)(t >> 32), k, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    palsgd_oracle_philox4x32_10(ctr, key, out);
    return out[0];
}

int palsgd_oracle_decision(uint64_t seed, uint64_t t, uint32_t k, double p)
{
    uint64_t r = (uint64_t)palsgd_oracle_draw_word(seed, t, k);
    return r < palsgd_oracle_threshold(p) ? 1 : 0;
}

/* ---- bfloat16 -------------------------------------------------------------- */

float palsgd_oracle_bf16_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* binary32 -> bfloat16, round to nearest, ties to even (NaN stays NaN). */
uint16_t palsgd_oracle_bf16_from_f32(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu) != 0u)
        return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t kept_lsb = (u >> 16) & 1u;
    uint32_t dropped  = u & 0xFFFFu;
    uint32_t top      = u >> 16;
    if (dropped > 0x8000u || (dropped == 0x8000u && kept_lsb))
        top += 1u;                      /* carries into the exponent correctly */
    return (uint16_t)top;
}

/* binary64 -> bfloat16 in ONE rounding (no double rounding through binary32).
 * bfloat16 has 8 significand bits and binary32's exponent range.             */
uint16_t palsgd_oracle_bf16_from_f64(double d)
{
    if (isnan(d)) return 0x7FC0u;
    uint16_t sign = signbit(d) ? 0x8000u : 0u;
    double a = fabs(d);
    if (a == 0.0) return sign;
    if (isinf(a)) return (uint16_t)(sign | 0x7F80u);
    int e;
    (void)frexp(a, &e);                 /* a = f * 2^e, f in [0.5, 1)          */
    int exp2 = e - 1;                   /* a in [2^exp2, 2^(exp2+1))           */
    if (exp2 < -126) exp2 = -126;       /* subnormal range: fixed quantum      */
    double q = ldexp(a, 7 - exp2);      /* quantum of bf16 at this binade = 1  */
    double r = nearbyint(q);            /* default mode: nearest, ties to even */
    float back = (float)ldexp(r, exp2 - 7);   /* exact: fits 8 bits            */
    if (isinf(back)) return (uint16_t)(sign | 0x7F80u);
    uint32_t u;
    memcpy(&u, &back, 4);
    return (uint16_t)(sign | (uint16_t)(u >> 16));
}

/* ---- global gradient norm ------------------------------------------------- */

/* The sum of squares behind a global-norm gradient clip, defined here as the
 * EXACT sum  sum_i g_i^2  rounded once to binary64.  It is realised with
 * binary128 arithmetic: every square of a binary32/binary64 value is exact in
 * binary128, and the accumulated rounding error of n additions (n * 2^-113
 * relative) is far below half a unit of binary64, so the result is the correctly
 * rounded exact sum except with negligible probability.  Because the sum is
 * exact, the order of the terms does not matter; the index range is split into
 * one contiguous block per thread and the block sums are added in block order.
 * Not re-entrant (one static table of block sums).                             */
#define SUMSQ_MAX_THREADS 1024
#define SUMSQ_BODY(LOAD)                                                        \
    static __float128 part[SUMSQ_MAX_THREADS];                                  \
    int used = 1;                                                               \
    _Pragma("omp parallel")                                                     \
    {                                                                           \
        int me = 0, nt = 1;                                                     \
        me = oracle_thread_id(); nt = oracle_thread_count();                    \
        if (nt > SUMSQ_MAX_THREADS) nt = SUMSQ_MAX_THREADS;                     \
        if (me == 0) used = nt;                                                 \
        if (me < nt) {                                                          \
            /* thread `me` sums the contiguous block [lo, hi) */                \
            uint64_t lo = n / (uint64_t)nt * (uint64_t)me;                      \
            uint64_t hi = me == nt - 1 ? n : n / (uint64_t)nt * (uint64_t)(me + 1); \
            __float128 acc = 0;                                                 \
            for (uint64_t i = lo; i < hi; ++i) {                                \
                __float128 x = (__float128)(LOAD);                              \
                acc += x * x;                                                   \
            }                                                                   \
            part[me] = acc;                                                     \
        }                                                                       \
    }                                                                           \
    __float128 total = 0;                                                       \
    for (int j = 0; j < used; ++j) total += part[j];                            \
    return (double)total;

double palsgd_oracle_sumsq_f32(const float *g, uint64_t n)     { SUMSQ_BODY(g[i]) }
double palsgd_oracle_sumsq_f64(const double *g, uint64_t n)    { SUMSQ_BODY(g[i]) }
double palsgd_oracle_sumsq_bf16(const uint16_t *g, uint64_t n) { SUMSQ_BODY(palsgd_oracle_bf16_to_f32(g[i])) }

/* Clip coefficient of a global-norm clip with threshold max_norm, in the
 * convention of the software the paper ran (PyTorch's clip_grad_norm_; the paper
 * only says that clipping was enabled, Appendix B):
 *     norm = sqrt(sumsq);  c = max_norm / (norm + 1e-6);  c = min(c, 1),
 * all in binary64.  The gradient is then multiplied by c.                       */
double palsgd_oracle_clip_coef(double sumsq, double max_norm)
{
    double norm = sqrt(sumsq);
    double c = max_norm / (norm + 1e-6);
    return c < 1.0 ? c : 1.0;
}

/* ---- learning-rate schedules ----------------------------------------------- */

/* Value at step t of a schedule with a linear warm-up followed by a constant
 * (kind 0) or by cosine annealing (kind 1), the form the paper's experiments use
 * for the outer learning rate (Appendix B):
 *   t <  warmup : base * (start_factor + (1 - start_factor) * t / warmup)
 *   t >= warmup : kind 0: base
 *                 kind 1: min + (base - min) * (1 + cos(pi * tau / (total - warmup))) / 2,
 *                         tau = min(t, total) - warmup           (stays at min after total) */
double palsgd_oracle_schedule(int kind, uint64_t t, uint64_t warmup, uint64_t total,
                              double base, double min_value, double start_factor)
{
    const double pi = 3.14159265358979323846;
    if (t < warmup)
        return base * (start_factor + (1.0 - start_factor) * (double)t / (double)warmup);
    if (kind == 0 || total <= warmup) return base;
    uint64_t tt = t < total ? t : total;
    double tau = (double)(tt - warmup);
    return min_value + (base - min_value) * (1.0 + cos(pi * tau / (double)(total - warmup))) / 2.0;
}

/* ---- thread count of the element loops (timing harness only) -------------- */
#ifdef _OPENMP
void palsgd_oracle_set_threads(int n) { if (n > 0) omp_set_num_threads(n); }
int  palsgd_oracle_get_threads(void)  { return omp_get_max_threads(); }
#else
void palsgd_oracle_set_threads(int n) { (void)n; }
int  palsgd_oracle_get_threads(void)  { return 1; }
#endif
