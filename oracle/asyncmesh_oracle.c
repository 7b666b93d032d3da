/*
 * asyncmesh_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, single-threaded CPU statement of the AsyncMesh per-step
 * parameter update for R data-parallel replicas x S pipeline stages.  It is
 * what the CUDA library is checked against; it shares no code with it and
 * nothing in the product path may call it.  Only the tests, the smoke check
 * and the benchmark's CPU-baseline leg load this file.
 *
 * What one step computes, per stage j, replica i, coordinate mu (paper
 * notation; m -> R replicas, P -> S stages):
 *
 *   O1  local optimizer step  w^_i^t = w_i^{t-1} - eta * update(g_i^{t-1})
 *       (first line of Eq. "sparta", Section 2.3).  The optimizer is the
 *       textbook decoupled-weight-decay Adam (AdamW) with bias correction;
 *       its moments m, v are local to a replica and never averaged.
 *       Alternatively NAdamW, the optimizer the paper itself uses for
 *       asynchronous pipelines (Appendix B.1: NAdamW, momentum 0.99): Adam with
 *       Nesterov momentum (Dozat, 2016) and decoupled weight decay.  With
 *       mu_t = beta1 (1 - 0.5 * 0.96^(t psi)) and PI_t = mu_1 ... mu_t:
 *           w^ = w - lr wd w - lr (1 - mu_t)/(1 - PI_t)        g / (sqrt(v^) + eps)
 *                            - lr mu_{t+1}/(1 - PI_t mu_{t+1}) m / (sqrt(v^) + eps)
 *       (m, v updated first; v^ bias-corrected, m is not: the momentum schedule
 *       takes that role).
 *   O2  snapshot of w^_i^t for the averaging launched at step t
 *       (Section 3.1: the average of step t arrives tau steps later; the
 *       appendix says the asynchronous setup is simulated by buffering).
 *       Here: a DENSE history of the last tau+1 full w^ vectors.
 *   O3  delayed sparse averaging with the EMA staleness estimate
 *       (Eq. "asparta", Eq. "ema" and the corrected-averaging equation that
 *       follows it, Section 3.2).  For mu in S^{t-tau}:
 *           wbar  = (1/R) sum_i w^_i^{t-tau}[mu]
 *           d_i  <- (1-lambda) d_i + lambda (w^_i^t[mu] - w^_i^{t-tau}[mu])
 *           w_i^t = wbar + d_i
 *       and w_i^t = w^_i^t for mu outside S^{t-tau}; d is untouched there.
 *       Nothing is consumed while t <= tau (no average has arrived yet).
 *       With an averaging interval K > 1 (end of Section 3.2: averaging "every K
 *       steps") O3 runs only at steps t = K, 2K, ...; the steps in between are
 *       purely local (w^t = w^).  tau is then a multiple of K, so the average
 *       consumed at a round was launched at an earlier round.
 *       The same paragraph names a second staleness estimate, that of eager
 *       DiLoCo, as a special case (all parameters, tau = K):
 *           d_i = (1/R) (w^_i^t[mu] - w^_i^{t-tau}[mu])
 *       selectable here for any p, tau, K (correction = 1); w_i^t = wbar + d_i
 *       as before.
 *   O4  pipeline look-ahead (Section 2.2): the last update direction
 *       (w^t - w^{t-1}) extrapolated by the stage's delay delta_j:
 *           look_i = w_i^t + delta_j (w_i^t - w_i^{t-1}).
 *
 * The random subset S_j^u (Section 2.3: one subset per stage, shared by its
 * replicas; Lemma 1: each element is in it independently with probability p)
 * is a counter-based rule: Philox-4x32-10 (Salmon et al., SC'11) with
 * key = (seed lo, seed hi), counter = (mu >> 2, j, (uint32) u, 0); coordinate
 * mu takes output word mu & 3 and is selected iff word < floor(p * 2^32).
 *
 * Arithmetic: fp32 storage, every operation a single IEEE-754 binary32
 * round-to-nearest operation in the order written (compile with
 * -ffp-contract=off, no -ffast-math).  Per-step scalars are formed in double
 * and rounded to float exactly once.
 *
 * Pins (tests, "not gpu"): published Philox known-answer vectors, AdamW
 * against torch.optim.AdamW and a closed form, the reductions tau=0 -> Eq.
 * "sparta", lambda=0 -> Eq. "asparta", lambda=1 -> raw difference, p=1,tau=0
 * -> full averaging, mean invariance, Lemma 1's (1-p) factor, a brute-force
 * trace written separately from the equations (also with an averaging interval,
 * with the bfloat16 / E4M3 exchange and with the eager estimate), chunk
 * independence; NAdamW against torch.optim.NAdam; the bfloat16 and E4M3 roundings
 * against the formats' definitions and the tensor library's casts; the eager
 * estimate against its closed form; the spread of d against numpy.
 * The look-ahead formula for delay > 0 is this build's reading of a sentence
 * (the paper prints no formula): PARITY UNPINNED beyond delay = 0 and the
 * constant-velocity closed form.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct am_oracle {
    uint32_t R, S, tau;
    uint32_t K;           /* averaging interval: subsets are exchanged at steps t = K, 2K, ... */
    uint32_t optimizer;   /* 0 AdamW, 1 NAdamW                                                  */
    uint32_t exchange;    /* 0: subsets exchanged in fp32; 1: rounded to bfloat16 on the wire;
                             2: rounded to 8-bit floating point (E4M3)                           */
    uint32_t correction;  /* 0: EMA staleness estimate (Eq. "ema"); 1: eager estimate
                             d_i = (w^_i^t - w^_i^{t-tau}) / R (end of Section 3.2)              */
    uint32_t stored;      /* 0: a replica remembers its own snapshot unrounded; 1: the snapshot
                             exists only as exchanged (see am_oracle_set_snapshot_storage)       */
    double momentum_decay, mu_product; /* NAdam's momentum schedule and its running product      */
    uint64_t *numel;      /* [S] coordinates held for stage j               */
    uint64_t *coord_base; /* [S] global index of local coordinate 0         */
    uint32_t *delay;      /* [S] look-ahead delay delta_j                   */
    double p, lambda, lr, beta1, beta2, eps, wd;
    uint64_t seed;
    uint64_t thresh;      /* floor(p * 2^32), in [0, 2^32]                  */
    uint64_t t;           /* steps taken                                    */
    float **w, **m, **v, **d, **wprev, **what, **look; /* [S] -> [R][numel] */
    float **H;            /* [S] -> [tau+1][R][numel] dense history of w^   */
} am_oracle;

/* ---- Philox-4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) ---------------- */

void am_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2],
                             uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* floor(p * 2^32) evaluated in double; p = 1 gives 2^32 (everything). */
uint64_t am_oracle_threshold(double p)
{
    return (uint64_t)floor(p * 4294967296.0);
}

/* Is global coordinate mu of stage j in the subset drawn for step u? */
int am_oracle_selected(uint64_t seed, uint64_t thresh, uint32_t stage,
                       uint64_t u, uint64_t mu)
{
    uint32_t ctr[4] = { (uint32_t)(mu >> 2), stage, (uint32_t)u, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t x[4];
    am_oracle_philox4x32_10(ctr, key, x);
    return (uint64_t)x[mu & 3] < thresh;
}

/* ---- life cycle --------------------------------------------------------- */

static float **alloc_rows(uint32_t S, const uint64_t *numel, uint64_t mult)
{
    float **a = (float **)calloc(S, sizeof(float *));
    if (!a) return NULL;
    for (uint32_t s = 0; s < S; ++s) {
        a[s] = (float *)calloc(numel[s] * mult, sizeof(float));
        if (!a[s]) return NULL;
    }
    return a;
}

static void free_rows(float **a, uint32_t S)
{
    if (!a) return;
    for (uint32_t s = 0; s < S; ++s) free(a[s]);
    free(a);
}

void am_oracle_destroy(am_oracle *o)
{
    if (!o) return;
    free_rows(o->w, o->S); free_rows(o->m, o->S); free_rows(o->v, o->S);
    free_rows(o->d, o->S); free_rows(o->wprev, o->S);
    free_rows(o->what, o->S); free_rows(o->look, o->S); free_rows(o->H, o->S);
    free(o->numel); free(o->coord_base); free(o->delay);
    free(o);
}

/*
 * coord_base may be NULL (all zero).  A non-zero base makes this instance
 * stand for coordinates [base, base + numel) of a larger stage: the subset
 * rule is evaluated at the global index, everything else is elementwise
 * (appendix, remark after Theorem 2), so a slice evolves exactly as it would
 * inside the full vector.  delay may be NULL (delta_j = S - 1 - j).
 */
am_oracle *am_oracle_create(uint32_t R, uint32_t S, const uint64_t *numel,
                            const uint64_t *coord_base, double p, uint32_t tau,
                            double lambda, double lr, double beta1,
                            double beta2, double eps, double wd, uint64_t seed,
                            const uint32_t *delay, uint32_t avg_interval)
{
    if (R < 1 || S < 1 || !numel || p < 0.0 || p > 1.0) return NULL;
    if (avg_interval < 1) avg_interval = 1;
    if (tau % avg_interval != 0) return NULL;
    am_oracle *o = (am_oracle *)calloc(1, sizeof(am_oracle));
    if (!o) return NULL;
    o->R = R; o->S = S; o->tau = tau; o->K = avg_interval;
    o->p = p; o->lambda = lambda; o->lr = lr; o->beta1 = beta1;
    o->beta2 = beta2; o->eps = eps; o->wd = wd; o->seed = seed;
    o->thresh = am_oracle_threshold(p);
    o->numel = (uint64_t *)calloc(S, sizeof(uint64_t));
    o->coord_base = (uint64_t *)calloc(S, sizeof(uint64_t));
    o->delay = (uint32_t *)calloc(S, sizeof(uint32_t));
    if (!o->numel || !o->coord_base || !o->delay) { am_oracle_destroy(o); return NULL; }
    for (uint32_t s = 0; s < S; ++s) {
        o->numel[s] = numel[s];
        o->coord_base[s] = coord_base ? coord_base[s] : 0;
        o->delay[s] = delay ? delay[s] : (S - 1 - s);
    }
    o->w = alloc_rows(S, numel, R);     o->m = alloc_rows(S, numel, R);
    o->v = alloc_rows(S, numel, R);     o->d = alloc_rows(S, numel, R);
    o->wprev = alloc_rows(S, numel, R); o->what = alloc_rows(S, numel, R);
    o->look = alloc_rows(S, numel, R);
    o->H = alloc_rows(S, numel, (uint64_t)R * (tau + 1));
    if (!o->w || !o->m || !o->v || !o->d || !o->wprev || !o->what ||
        !o->look || !o->H) { am_oracle_destroy(o); return NULL; }
    return o;
}

/* Set the initial weights of one replica (replica < 0: all replicas, the
 * homogeneous "same initialisation" of Section 3.3).  w^{-1} := w^0, so the
 * look-ahead before the first step is w^0 itself. */
int am_oracle_init_params(am_oracle *o, uint32_t stage, int32_t replica,
                          const float *src, uint64_t n)
{
    if (!o || stage >= o->S || n != o->numel[stage] || replica >= (int32_t)o->R)
        return -1;
    for (uint32_t i = 0; i < o->R; ++i) {
        if (replica >= 0 && (uint32_t)replica != i) continue;
        memcpy(o->w[stage] + (uint64_t)i * n, src, n * sizeof(float));
        memcpy(o->wprev[stage] + (uint64_t)i * n, src, n * sizeof(float));
        memcpy(o->look[stage] + (uint64_t)i * n, src, n * sizeof(float));
    }
    return 0;
}

/* ---- one step ------------------------------------------------------------ */

/*
 * What a replica's snapshot value looks like to the others.  The paper's
 * quantisation study (Section 5.3, paragraph "Robustness of Sparse Averaging";
 * Appendix B.2) sends the subset in
 * reduced precision; with exchange = 1 every value entering the average is
 * first rounded to bfloat16 (round to nearest even: keep the upper 16 bits of
 * the binary32 pattern), with exchange = 2 to 8-bit floating point (E4M3, the
 * paper does not say which 8-bit format or scaling it used: plain cast, no
 * scale); the average itself is formed in fp32, and a replica's own staleness
 * sample still uses its own unrounded value, which never left it.
 */
/*
 * Nearest value of the 8-bit floating-point format E4M3 (4 exponent bits, bias 7,
 * 3 mantissa bits, no infinities, largest finite value 448): ties to even,
 * magnitudes above 448 clamp to 448, the spacing below 2^-6 is 2^-9 (subnormals).
 */
static float round_e4m3(float x)
{
    if (isnan(x)) return x;
    float a = fabsf(x);
    if (a > 448.0f) a = 448.0f;
    if (a == 0.0f) return x;
    int e;
    (void)frexpf(a, &e);              /* a = f * 2^e with f in [0.5, 1): binade exponent e - 1 */
    int q = (e - 1) - 3;              /* exponent of the spacing: three mantissa bits         */
    if (q < -9) q = -9;               /* subnormal range                                      */
    float r = ldexpf(nearbyintf(ldexpf(a, -q)), q);   /* nearbyintf: ties to even             */
    if (r > 448.0f) r = 448.0f;
    return copysignf(r, x);
}

static float exchanged(const am_oracle *o, float x)
{
    if (o->exchange == 0) return x;
    if (o->exchange == 2) return round_e4m3(x);
    uint32_t u;
    memcpy(&u, &x, sizeof u);
    if ((u & 0x7F800000u) != 0x7F800000u)          /* finite: round to nearest even */
        u += 0x7FFFu + ((u >> 16) & 1u);
    u &= 0xFFFF0000u;
    memcpy(&x, &u, sizeof x);
    return x;
}

void am_oracle_set_exchange(am_oracle *o, uint32_t exchange)
{
    if (o) o->exchange = exchange;
}

void am_oracle_set_correction(am_oracle *o, uint32_t correction)
{
    if (o) o->correction = correction;
}

/*
 * Second reading of the reduced-precision exchange (Section 5.3, paragraph
 * "Robustness of Sparse Averaging"; Appendix B.2): the paper does not say whether a
 * replica keeps an unrounded copy of what it sent.  stored = 0 (default): it does,
 * and its staleness sample w^_i^t - w^_i^{t-tau} uses that copy.  stored = 1: the
 * snapshot exists only in the exchanged precision, for its owner too, so the sample
 * is taken against the rounded value and the snapshot memory shrinks with the format.
 */
void am_oracle_set_snapshot_storage(am_oracle *o, uint32_t stored)
{
    if (o) o->stored = stored;
}

float am_oracle_exchanged(uint32_t exchange, float x)
{
    am_oracle tmp;
    memset(&tmp, 0, sizeof tmp);
    tmp.exchange = exchange;
    return exchanged(&tmp, x);
}

/*
 * grads[j] points to [R][numel_j] floats, row i = gradient of replica i.
 * lambda_t / lr_t < 0 mean "use the constant given at creation"; otherwise
 * they replace it for this step (the paper decays both over training).
 */
void am_oracle_set_optimizer(am_oracle *o, uint32_t optimizer, double momentum_decay)
{
    if (!o) return;
    o->optimizer = optimizer;
    o->momentum_decay = momentum_decay;
    o->mu_product = 1.0;
}

int am_oracle_step_ex(am_oracle *o, const float *const *grads, double lambda_t,
                      double lr_t)
{
    if (!o || !grads) return -1;
    const uint64_t t = ++o->t;
    const uint32_t R = o->R, tau = o->tau;
    const double lam_d = lambda_t >= 0.0 ? lambda_t : o->lambda;
    const double lr_d = lr_t >= 0.0 ? lr_t : o->lr;

    /* per-step scalars: double arithmetic, one rounding to float each */
    const float b1 = (float)o->beta1, b2 = (float)o->beta2;
    const float omb1 = (float)(1.0 - o->beta1), omb2 = (float)(1.0 - o->beta2);
    const float ib1 = (float)(1.0 / (1.0 - pow(o->beta1, (double)t)));
    const float ib2 = (float)(1.0 / (1.0 - pow(o->beta2, (double)t)));
    const float lr = (float)lr_d, lrwd = (float)(lr_d * o->wd);
    const float eps = (float)o->eps;
    const float lam = (float)lam_d, oml = (float)(1.0 - lam_d);
    const float Rf = (float)R;
    /* NAdam's momentum schedule (scalars only; unused by AdamW) */
    const double mu_t = o->beta1 * (1.0 - 0.5 * pow(0.96, (double)t * o->momentum_decay));
    const double mu_n = o->beta1 * (1.0 - 0.5 * pow(0.96, (double)(t + 1) * o->momentum_decay));
    if (o->mu_product == 0.0) o->mu_product = 1.0;
    o->mu_product *= mu_t;
    const float cg = (float)(lr_d * (1.0 - mu_t) / (1.0 - o->mu_product));
    const float cm = (float)(lr_d * mu_n / (1.0 - o->mu_product * mu_n));

    for (uint32_t s = 0; s < o->S; ++s) {
        const uint64_t N = o->numel[s];
        float *w = o->w[s], *m = o->m[s], *v = o->v[s], *d = o->d[s];
        float *wprev = o->wprev[s], *what = o->what[s], *look = o->look[s];
        const float *g = grads[s];
        float *Hnow = o->H[s] + (t % (tau + 1)) * (uint64_t)R * N;

        /* O1 + O2: AdamW on every replica, snapshot of the local result */
        for (uint32_t i = 0; i < R; ++i) {
            for (uint64_t mu = 0; mu < N; ++mu) {
                const uint64_t k = (uint64_t)i * N + mu;
                const float gk = g[k];
                const float mk = (b1 * m[k]) + (omb1 * gk);
                const float vk = (b2 * v[k]) + (omb2 * (gk * gk));
                m[k] = mk;
                v[k] = vk;
                const float mh = mk * ib1;
                const float vh = vk * ib2;
                const float den = sqrtf(vh) + eps;
                const float wk = w[k];
                float wh = wk - (lrwd * wk);   /* decoupled weight decay */
                if (o->optimizer == 0) {
                    const float u = mh / den;
                    wh = wh - (lr * u);        /* Adam step              */
                } else {
                    const float ug = gk / den; /* Nesterov: gradient part ... */
                    const float um = mk / den; /* ... and momentum part       */
                    wh = wh - (cg * ug);
                    wh = wh - (cm * um);
                }
                wprev[k] = wk;
                what[k] = wh;
                Hnow[k] = o->stored ? exchanged(o, wh) : wh;
            }
        }

        /* O3: delayed sparse averaging with EMA staleness correction */
        const int consuming = (t % o->K == 0) && t > tau;   /* an averaging round with an arrival */
        const uint64_t u_step = t - tau;   /* only meaningful if consuming */
        const float *Hold = o->H[s] + (u_step % (tau + 1)) * (uint64_t)R * N;
        for (uint64_t mu = 0; mu < N; ++mu) {
            int sel = 0;
            if (consuming)
                sel = am_oracle_selected(o->seed, o->thresh, s, u_step,
                                         o->coord_base[s] + mu);
            if (sel) {
                float a = exchanged(o, Hold[mu]);
                for (uint32_t i = 1; i < R; ++i)
                    a = a + exchanged(o, Hold[(uint64_t)i * N + mu]);
                const float abar = a / Rf;
                for (uint32_t i = 0; i < R; ++i) {
                    const uint64_t k = (uint64_t)i * N + mu;
                    const float diff = what[k] - Hold[k];
                    float dk;
                    if (o->correction == 0)
                        dk = (oml * d[k]) + (lam * diff);   /* Eq. "ema"          */
                    else
                        dk = diff / Rf;                     /* eager estimate     */
                    d[k] = dk;
                    w[k] = abar + dk;
                }
            } else {
                for (uint32_t i = 0; i < R; ++i) {
                    const uint64_t k = (uint64_t)i * N + mu;
                    w[k] = what[k];
                }
            }
        }

        /* O4: look-ahead by the stage's delay.  With delay 0 nothing is
         * extrapolated: the look-ahead weights ARE the current weights (the
         * product w + 0 * (w - w_prev) is not that for w = +-Inf, where it is
         * NaN, nor for w = -0, where it is +0). */
        const float delta = (float)o->delay[s];
        for (uint64_t k = 0; k < (uint64_t)R * N; ++k) {
            const float dir = w[k] - wprev[k];
            look[k] = o->delay[s] == 0 ? w[k] : w[k] + (delta * dir);
        }
    }
    return 0;
}

int am_oracle_step(am_oracle *o, const float *const *grads)
{
    return am_oracle_step_ex(o, grads, -1.0, -1.0);
}

/* ---- read-back ----------------------------------------------------------- */

/* which: 0 w, 1 m, 2 v, 3 d, 4 look, 5 w^ (pre-averaging), 6 w^{t-1}.
 * replica in [0, R).  Returns a pointer to numel[stage] floats. */
const float *am_oracle_row(const am_oracle *o, uint32_t stage, int which,
                           uint32_t replica)
{
    if (!o || stage >= o->S || replica >= o->R) return NULL;
    float **a = NULL;
    switch (which) {
    case 0: a = o->w; break;     case 1: a = o->m; break;
    case 2: a = o->v; break;     case 3: a = o->d; break;
    case 4: a = o->look; break;  case 5: a = o->what; break;
    case 6: a = o->wprev; break; default: return NULL;
    }
    return a[stage] + (uint64_t)replica * o->numel[stage];
}

/* Look-ahead weights of a stage for any delay (Section 2.2): the same
 * extrapolation as O4, w + delay (w - w^{t-1}), from the current and the
 * previous weights.  dst receives [R][numel] floats. */
int am_oracle_lookahead(const am_oracle *o, uint32_t stage, uint32_t delay, float *dst)
{
    if (!o || stage >= o->S || !dst) return -1;
    const uint64_t n = (uint64_t)o->R * o->numel[stage];
    const float delta = (float)delay;
    for (uint64_t k = 0; k < n; ++k) {
        const float dir = o->w[stage][k] - o->wprev[stage][k];
        dst[k] = delay == 0 ? o->w[stage][k] : o->w[stage][k] + (delta * dir);   /* delay 0: w itself */
    }
    return 0;
}

/* Replica mean of the weights (the consensus model the paper evaluates):
 * sequential sum over i = 0..R-1, one division by (float) R. */
int am_oracle_mean_params(const am_oracle *o, uint32_t stage, float *dst)
{
    if (!o || stage >= o->S || !dst) return -1;
    const uint64_t N = o->numel[stage];
    const float Rf = (float)o->R;
    for (uint64_t mu = 0; mu < N; ++mu) {
        float a = o->w[stage][mu];
        for (uint32_t i = 1; i < o->R; ++i)
            a = a + o->w[stage][(uint64_t)i * N + mu];
        dst[mu] = a / Rf;
    }
    return 0;
}

/* Consensus error of Section 3.3: sum_i ||w_i - wbar||^2 over the stage,
 * accumulated in double from the fp32 weights. */
double am_oracle_consensus_error(const am_oracle *o, uint32_t stage)
{
    if (!o || stage >= o->S) return -1.0;
    const uint64_t N = o->numel[stage];
    double acc = 0.0;
    for (uint64_t mu = 0; mu < N; ++mu) {
        double mean = 0.0;
        for (uint32_t i = 0; i < o->R; ++i)
            mean += (double)o->w[stage][(uint64_t)i * N + mu];
        mean /= (double)o->R;
        for (uint32_t i = 0; i < o->R; ++i) {
            const double e = (double)o->w[stage][(uint64_t)i * N + mu] - mean;
            acc += e * e;
        }
    }
    return acc;
}

/* Spread of the staleness estimates across replicas (the appendix figure on the
 * consensus error plots the "variance between EMA estimates in each replica",
 * mean and max across the model dimension): per coordinate the population
 * variance (1/R) sum_i (d_i - dbar)^2 in double; *mean_out = its mean over the
 * stage's coordinates, *max_out = its maximum. */
int am_oracle_ema_variance(const am_oracle *o, uint32_t stage, double *mean_out,
                           double *max_out)
{
    if (!o || stage >= o->S || !mean_out || !max_out) return -1;
    const uint64_t N = o->numel[stage];
    double sum = 0.0, mx = 0.0;
    for (uint64_t mu = 0; mu < N; ++mu) {
        double mean = 0.0;
        for (uint32_t i = 0; i < o->R; ++i)
            mean += (double)o->d[stage][(uint64_t)i * N + mu];
        mean /= (double)o->R;
        double var = 0.0;
        for (uint32_t i = 0; i < o->R; ++i) {
            const double e = (double)o->d[stage][(uint64_t)i * N + mu] - mean;
            var += e * e;
        }
        var /= (double)o->R;
        sum += var;
        if (var > mx) mx = var;
    }
    *mean_out = sum / (double)N;
    *max_out = mx;
    return 0;
}

/* One byte (0/1) per local coordinate: membership in S_stage^u. */
int am_oracle_subset_mask(const am_oracle *o, uint32_t stage, uint64_t u,
                          uint8_t *mask)
{
    if (!o || stage >= o->S || !mask) return -1;
    for (uint64_t mu = 0; mu < o->numel[stage]; ++mu)
        mask[mu] = (uint8_t)am_oracle_selected(o->seed, o->thresh, stage, u,
                                               o->coord_base[stage] + mu);
    return 0;
}

uint64_t am_oracle_step_count(const am_oracle *o) { return o ? o->t : 0; }
