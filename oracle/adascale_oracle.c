/*
 * AdaScale gain-ratio step: CPU oracle.
 *
 * TEST INFRASTRUCTURE, NOT PRODUCT CODE.  This file is the plain, slow, fp64
 * statement of what one AdaScale iteration computes, written from the paper
 * (Johnson, Agrawal, Gu, Guestrin: "AdaScale SGD", ICML 2020).  It shares no
 * code, header, table or constant with the CUDA library and must never be
 * linked into, imported by or called from it.  Only the tests, the smoke
 * check and the benchmark's CPU-baseline leg may use it.
 *
 * What is written out here, in the paper's order and notation:
 *   - Sec. 2 ("scaled SGD"): the S per-batch gradients g^(1..S) are averaged
 *     into gbar.
 *   - App. B.3: sigma_hat^2 = 1/(S-1) sum_i ||g^(i)||^2 - S/(S-1) ||gbar||^2 and
 *     mu_hat^2 = ||gbar||^2 - sigma_hat^2 / S, the clamps max(sigma_hat^2, eps)
 *     and max(mu_hat^2, 0), the moving averages with parameter theta and
 *     the plain-mean warm start.
 *   - Eq. 3 with the averages plugged in: r = (s + m) / (s/S + m).
 *   - Sec. 3.2: eta_t = r_t * lr(floor(tau_t)), tau_{t+1} = tau_t + r_t.
 *   - App. B.1: the exponential-decay and step-decay families of lr.
 *   - Sec. 3.4: the alternative estimator r_hat = (m1+eps)/(m2+eps).
 *   - Eq. 2 with momentum (Sec. 3.4): the parameter update.
 *
 * sigma_hat^2 is evaluated as the sum over coordinates of the textbook two-pass
 * sample variance of the S values of that coordinate (Sec. 3.1 defines the
 * variance as the sum of the per-entry variances; dividing the summed squared
 * deviations by S-1 is algebraically the formula of App. B.3).  The raw sum
 * Q = sum_i ||g^(i)||^2 is returned as well so that a test can evaluate the
 * formula exactly as the paper prints it.
 *
 * Readings where the paper is silent (each pinned or marked in the tests):
 *   - moving average: xbar <- th*xbar + (1-th)*xhat, th = min(theta, 1 - 1/n),
 *     n = samples absorbed including this one (a plain mean while n < 1/(1-theta));
 *   - mu_hat^2 is formed from the unclamped sigma_hat^2, both are clamped after;
 *   - momentum: v <- rho v + (gbar + lambda w); w <- w - eta v.   PARITY UNPINNED
 *     by the paper (it says only "momentum-SGD" and "weight decay"); the
 *     arithmetic of this reading is pinned by its geometric-series closed form
 *     and by rho = 0, lambda = 0 reducing to Eq. 2;
 *   - S = 1: r = 1 (App. A.2), statistics skipped;
 *   - non-finite sums: PARITY UNPINNED extension; the step is skipped (no state
 *     change, eta = 0) and a flag is raised.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };
enum { ORACLE_LR_CONST = 0, ORACLE_LR_EXP = 1, ORACLE_LR_STEP = 2 };
enum { ORACLE_FLAG_LAGGED = 1, ORACLE_FLAG_CONT_TAU = 2, ORACLE_FLAG_RATIO = 4 };

typedef struct {
    int kind;
    double eta0; /* eta_0 */
    double d;    /* decay factor d */
    double T_S1; /* total iterations at scale 1 (exponential family) */
    int n;       /* number of step boundaries w_i */
    double w[8]; /* step boundaries w_i */
} oracle_lr;

typedef struct {
    int S;
    double eps;   /* epsilon of the clamp / of the ratio estimator */
    double theta; /* moving-average parameter; < 0 selects max(1 - S/1000, 0) */
    int flags;
} oracle_cfg;

typedef struct {
    /* persistent */
    double tau;    /* scale-invariant iteration tau_t */
    double avg_a;  /* sigma_bar^2   (ratio form: m1) */
    double avg_b;  /* mu_bar^2      (ratio form: m2) */
    long long n;   /* samples absorbed by the averages */
    long long t;   /* iterations applied */
    long long skipped;
    /* results of the most recent step */
    double r, eta, lr;
    double sigma2_raw, mu2_raw; /* before the clamps */
    double sigma2_hat, mu2_hat; /* after the clamps  */
    int nonfinite;
} oracle_state;

/* App. B.1: lr(t) = eta0 * d^(t / T_S1)  or  eta0 * d^(#{i : t > w_i}). */
double oracle_lr_eval(const oracle_lr *lr, double t)
{
    if (lr->kind == ORACLE_LR_EXP)
        return lr->eta0 * pow(lr->d, t / lr->T_S1);
    if (lr->kind == ORACLE_LR_STEP) {
        int count = 0;
        for (int i = 0; i < lr->n; ++i)
            if (t > lr->w[i])
                count += 1;
        return lr->eta0 * pow(lr->d, (double)count);
    }
    return lr->eta0;
}

/* App. B.3 / Sec. 3.4: theta = max{1 - S/1000, 0} unless the caller fixes it. */
double oracle_theta(const oracle_cfg *cfg)
{
    if (cfg->theta >= 0.0)
        return cfg->theta;
    double th = 1.0 - (double)cfg->S / 1000.0;
    return th > 0.0 ? th : 0.0;
}

static double load_elem(const void *row, long long j, int dtype)
{
    if (dtype == ORACLE_BF16) {
        uint32_t bits = (uint32_t)((const uint16_t *)row)[j] << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return (double)((const float *)row)[j];
}

/*
 * Columns [0, n) of S rows.  Adds to *D the summed squared deviations
 * sum_j sum_i (g_ij - gbar_j)^2, to *N the squared norm sum_j gbar_j^2 and to *Q
 * the raw sum_j sum_i g_ij^2; writes gbar_j when gbar != NULL.  The caller
 * zeroes D, N, Q before the first range.
 */
void oracle_grad_stats(const void *const *rows, int S, long long n, int dtype, double *gbar,
                       double *D, double *N, double *Q, int nthreads)
{
    double d = 0.0, nn = 0.0, q = 0.0;
    if (nthreads < 1)
        nthreads = 1;
#pragma omp parallel for reduction(+ : d, nn, q) schedule(static) num_threads(nthreads)
    for (long long j = 0; j < n; ++j) {
        double sum = 0.0;
        for (int i = 0; i < S; ++i)
            sum += load_elem(rows[i], j, dtype);
        double mean = sum / (double)S;
        double dev = 0.0, raw = 0.0;
        for (int i = 0; i < S; ++i) {
            double g = load_elem(rows[i], j, dtype);
            dev += (g - mean) * (g - mean);
            raw += g * g;
        }
        if (gbar)
            gbar[j] = mean;
        d += dev;
        nn += mean * mean;
        q += raw;
    }
    *D += d;
    *N += nn;
    *Q += q;
}

static double moving_average(double prev, double sample, double theta, long long n)
{
    double th = 1.0 - 1.0 / (double)n; /* plain mean of the first n samples */
    if (theta < th)
        th = theta;
    return th * prev + (1.0 - th) * sample;
}

/* Eq. 3 with the averages in place of the expectations. */
static double gain_from_averages(double s, double m, int S)
{
    return (s + m) / (s / (double)S + m);
}

/*
 * One iteration's scalar work, given D, N, Q of this iteration's gradients.
 * Order: estimates -> clamps -> averages -> r_t -> eta_t from tau_t -> tau_{t+1}.
 */
void oracle_scalar_step(oracle_state *st, const oracle_cfg *cfg, const oracle_lr *lr, double D,
                        double N, double Q)
{
    const int S = cfg->S;
    const double theta = oracle_theta(cfg);
    st->nonfinite = 0;

    if (!isfinite(D) || !isfinite(N) || !isfinite(Q)) {
        st->nonfinite = 1;
        st->skipped += 1;
        st->eta = 0.0;
        return;
    }

    double t_arg = (cfg->flags & ORACLE_FLAG_CONT_TAU) ? st->tau : floor(st->tau);
    double r;

    if (S == 1) {
        /* App. A.2: at S = 1 the gain is 1 in every iteration. */
        st->sigma2_raw = 0.0;
        st->mu2_raw = N;
        st->sigma2_hat = 0.0;
        st->mu2_hat = N;
        r = 1.0;
    } else if (cfg->flags & ORACLE_FLAG_RATIO) {
        /* Sec. 3.4: m1 averages (1/S) sum_i ||g_i||^2, m2 averages ||gbar||^2. */
        double s1 = Q / (double)S, s2 = N;
        st->sigma2_raw = st->sigma2_hat = s1;
        st->mu2_raw = st->mu2_hat = s2;
        double r_prior = st->n > 0 ? (st->avg_a + cfg->eps) / (st->avg_b + cfg->eps) : 1.0;
        st->n += 1;
        st->avg_a = moving_average(st->avg_a, s1, theta, st->n);
        st->avg_b = moving_average(st->avg_b, s2, theta, st->n);
        r = (cfg->flags & ORACLE_FLAG_LAGGED) ? r_prior
                                              : (st->avg_a + cfg->eps) / (st->avg_b + cfg->eps);
    } else {
        /* App. B.3 */
        double sigma2 = D / (double)(S - 1);
        double mu2 = N - sigma2 / (double)S;
        st->sigma2_raw = sigma2;
        st->mu2_raw = mu2;
        if (sigma2 < cfg->eps)
            sigma2 = cfg->eps;
        if (mu2 < 0.0)
            mu2 = 0.0;
        st->sigma2_hat = sigma2;
        st->mu2_hat = mu2;
        /* r_0 = 1; later lagged gains use the averages of prior iterations only */
        double r_prior = st->n > 0 ? gain_from_averages(st->avg_a, st->avg_b, S) : 1.0;
        st->n += 1;
        st->avg_a = moving_average(st->avg_a, sigma2, theta, st->n);
        st->avg_b = moving_average(st->avg_b, mu2, theta, st->n);
        r = (cfg->flags & ORACLE_FLAG_LAGGED) ? r_prior
                                              : gain_from_averages(st->avg_a, st->avg_b, S);
    }

    st->r = r;
    st->lr = oracle_lr_eval(lr, t_arg);
    st->eta = r * st->lr;     /* Sec. 3.2: eta_t = r_t lr(floor(tau_t)) */
    st->tau = st->tau + r;    /* tau_{t+1} = tau_t + r_t */
    st->t += 1;
}

/* Momentum form of Eq. 2: v <- rho v + (gbar + lambda w); w <- w - eta v. */
void oracle_update(const double *gbar, double *w, double *v, long long n, double rho,
                   double lambda, double eta, int nthreads)
{
    if (nthreads < 1)
        nthreads = 1;
#pragma omp parallel for schedule(static) num_threads(nthreads)
    for (long long j = 0; j < n; ++j) {
        double vj = rho * v[j] + (gbar[j] + lambda * w[j]);
        v[j] = vj;
        w[j] = w[j] - eta * vj;
    }
}
