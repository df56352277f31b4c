/*
 * CPU oracle for the IMPACT learner loss and its circular buffer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * paper's learner computes per batch; it exists so that the CUDA library can be
 * checked against it.  It shares no code, header, table or constant with the CUDA
 * path and nothing in the product imports, links or runs it.
 *
 * Arithmetic: every input is read exactly as stored (fp32) and widened to fp64;
 * all arithmetic, including the sums over the batch, is serial fp64.
 *
 * Each function cites the passage of the paper it follows (IMPACT, arXiv 1912.00167).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    double vf_coef;    /* value-function coefficient (Appendix B tables) */
    double ent_coef;   /* entropy coefficient (Appendix B tables) */
    double kl_coef;    /* eta of Algorithm 1's KL term */
    double lambda;     /* lambda of V-trace GAE-lambda (Section 3.1) */
    double rho_tw;     /* rho of the target-worker clipping (Section 3.1), beta = 1/rho */
    int32_t is_source; /* 0: pi_target/pi_worker (Section 3.1); 1: pi_theta/pi_worker (Section 2.2);
                          2: no importance weights, rho = c = 1 (GAE-lambda as PPO uses it, Section 2.1) */
    int32_t ratio_mode;/* 0: R3, 1: R1, 2: R2 (Section 4.1) */
    int32_t objective; /* 0: epsilon-clipped surrogate (Appendix E); 1: IMPALA's importance-weighted
                          policy gradient with V-trace targets (Section 2.2, Appendix D) */
} oracle_coef;

/* log-softmax of one row: log pi(k|s) = z_k - log sum_j exp(z_j), max-shifted. */
static void log_softmax_row(const float* z, int64_t A, double* lp) {
    double m = (double)z[0];
    for (int64_t k = 1; k < A; ++k)
        if ((double)z[k] > m) m = (double)z[k];
    double s = 0.0;
    for (int64_t k = 0; k < A; ++k) s += exp((double)z[k] - m);
    double lse = m + log(s);
    for (int64_t k = 0; k < A; ++k) lp[k] = (double)z[k] - lse;
}

/*
 * Steps shared by the categorical and the Gaussian loss once the three
 * log-probabilities of the taken action are known, for ONE trajectory of T steps.
 *
 *  - truncated importance weights rho_t, c_t (Section 2.2; Section 3.1 for the
 *    target/worker form),
 *  - importance-sampled 1-step TD error delta_t V (Section 2.2, inside the V-trace sum),
 *  - V-trace GAE-lambda advantage (Section 3.1), written as its backward recursion
 *    A_t = delta_t + lambda * gamma_t * c_t * A_{t+1}, A_T = 0,
 *  - value target V_t + A_t (Algorithm 1's value gradient; equals the V-trace target of
 *    Section 2.2 when lambda = 1),
 *  - ratio R_t of Section 4.1 (R3 = pi_theta / max(pi_target, pi_worker / rho), Section 3.1)
 *    and the epsilon-clipped surrogate of Appendix E,
 *  - whether the gradient passes the clip (it does unless R lies strictly beyond the
 *    bound on the side where the clipped branch is the smaller one),
 *  - adv_cond: sum of the absolute values of the terms that make up A_t (a conditioning
 *    figure for the tests, no part of the loss).
 *
 * gamma_t = discounts[t] is the per-step discount, 0 where the episode ended at t.
 */
static void trajectory_terms(const double* lth, const double* ltg, const float* worker_logp,
                             const float* rewards, const float* discounts, const float* values,
                             double bootstrap, double rho_bar, double c_bar, double clip_eps,
                             const oracle_coef* cf, int64_t T, const int8_t* flip,
                             double* adv, double* vtarget, double* ratio, double* surr,
                             double* pass, double* rho_trunc, double* adv_cond, double* pgw) {
    double next_adv = 0.0, next_cond = 0.0;
    for (int64_t t = T - 1; t >= 0; --t) {
        double lw = (double)worker_logp[t];
        double x = (cf->is_source == 1 ? lth[t] : ltg[t]) - lw;
        double w = (cf->is_source == 2) ? 1.0 : exp(x);
        double rho = w < rho_bar ? w : rho_bar;
        double c = w < c_bar ? w : c_bar;
        double v = (double)values[t];
        double v_next = (t == T - 1) ? bootstrap : (double)values[t + 1];
        double g = (double)discounts[t];
        double delta = rho * ((double)rewards[t] + g * v_next - v);
        double a = delta + cf->lambda * g * c * next_adv;
        adv[t] = a;
        vtarget[t] = v + a;
        rho_trunc[t] = (w > rho_bar) ? 1.0 : 0.0;
        /* the same recursion on absolute values: the sum of |terms| of A_t, i.e. how much
         * cancellation A_t hides.  Not part of the loss; tests scale their tolerance by it. */
        next_cond = rho * (fabs((double)rewards[t]) + fabs(g * v_next) + fabs(v)) +
                    fabs(cf->lambda * g * c) * next_cond;
        adv_cond[t] = next_cond;
        next_adv = a;
        pgw[t] = rho; /* kept for the policy-gradient objective below */
    }
    if (cf->objective == 1) {
        /* IMPALA's actor update (Section 2.2; Appendix D calls it an importance-sampled vanilla
         * policy gradient): ascend rho_t (r_t + gamma_t v_{t+1} - V(s_t)) grad log pi_theta(a_t|s_t),
         * v the V-trace target (the bootstrap value after the last stored step).  The weight is a
         * constant for the gradient; the reported objective is weight * log pi_theta. */
        for (int64_t t = 0; t < T; ++t) {
            double v_next = (t == T - 1) ? bootstrap : vtarget[t + 1];
            double wgt = pgw[t] * ((double)rewards[t] + (double)discounts[t] * v_next - (double)values[t]);
            ratio[t] = pgw[t];
            pgw[t] = wgt;
            surr[t] = wgt * lth[t];
            pass[t] = 1.0;
        }
        return;
    }
    for (int64_t t = 0; t < T; ++t) {
        double lw = (double)worker_logp[t];
        double d;
        if (cf->ratio_mode == 1) d = ltg[t];
        else if (cf->ratio_mode == 2) d = lw;
        else {
            double alt = lw - log(cf->rho_tw);
            d = ltg[t] > alt ? ltg[t] : alt;
        }
        double R = exp(lth[t] - d);
        double lo = 1.0 - clip_eps, hi = 1.0 + clip_eps;
        double Rc = R < lo ? lo : (R > hi ? hi : R);
        double u = R * adv[t], cl = Rc * adv[t];
        surr[t] = u < cl ? u : cl;
        int clipped = (adv[t] > 0.0 && R > hi) || (adv[t] < 0.0 && R < lo);
        if (flip && flip[t]) clipped = !clipped;
        pass[t] = clipped ? 0.0 : 1.0;
        ratio[t] = R;
        pgw[t] = pass[t] * adv[t] * R;
    }
}

/*
 * Categorical IMPACT loss and gradients for a batch [B, T] with A actions.
 *
 * loss_terms[8] = { total, policy loss = -mean surrogate, value loss = mean 1/2 (V - Vhat)^2,
 *                   mean entropy of pi_theta, mean KL(pi_target || pi_theta),
 *                   fraction of steps whose gradient the epsilon-clip removed,
 *                   fraction of steps whose importance weight exceeded rho_bar, mean R }
 * total = policy + vf_coef * value - ent_coef * entropy + kl_coef * KL  (Algorithm 1, with
 * the 1/M normaliser over all M = B*T steps).
 *
 * dlogits, dvalues: gradient of `total` with the advantage and the value target held
 * constant (Algorithm 1 differentiates neither).  Optional outputs may be NULL.
 * `flip` (optional, [B,T]) inverts the clip decision of the marked steps; tests use it
 * to accept either branch where R sits on a clip bound to rounding.
 * Returns 0, or -1 on a bad argument.
 */
int oracle_impact_loss_categorical(
    const float* learner_logits, const float* target_logits, const float* worker_logp,
    const int32_t* actions, const float* rewards, const float* discounts,
    const float* values, const float* bootstrap_values,
    double rho_bar, double c_bar, double clip_eps, const oracle_coef* cf,
    int64_t B, int64_t T, int64_t A, const int8_t* flip,
    double* loss_terms, double* dlogits, double* dvalues,
    double* vtarget_out, double* advantage_out, double* ratio_out, double* adv_cond_out,
    double* pg_weight_out) {
    if (B <= 0 || T <= 0 || A <= 0 || !cf) return -1;
    const double M = (double)B * (double)T;
    double* lp_th = (double*)malloc(sizeof(double) * (size_t)(T * A));
    double* lp_tg = (double*)malloc(sizeof(double) * (size_t)(T * A));
    double* buf = (double*)malloc(sizeof(double) * (size_t)(T * 10));
    if (!lp_th || !lp_tg || !buf) { free(lp_th); free(lp_tg); free(buf); return -1; }
    double *lth = buf, *ltg = buf + T, *adv = buf + 2 * T, *vt = buf + 3 * T,
           *ratio = buf + 4 * T, *surr = buf + 5 * T, *pass = buf + 6 * T, *rtr = buf + 7 * T,
           *cond = buf + 8 * T, *pgw = buf + 9 * T;
    double s_surr = 0, s_val = 0, s_ent = 0, s_kl = 0, s_clip = 0, s_trunc = 0, s_ratio = 0;

    for (int64_t b = 0; b < B; ++b) {
        const float* zl = learner_logits + b * T * A;
        const float* zt = target_logits + b * T * A;
        const int32_t* act = actions + b * T;
        for (int64_t t = 0; t < T; ++t) {
            log_softmax_row(zl + t * A, A, lp_th + t * A);
            log_softmax_row(zt + t * A, A, lp_tg + t * A);
            int32_t a = act[t];
            if (a < 0 || a >= A) { free(lp_th); free(lp_tg); free(buf); return -1; }
            lth[t] = lp_th[t * A + a];
            ltg[t] = lp_tg[t * A + a];
        }
        trajectory_terms(lth, ltg, worker_logp + b * T, rewards + b * T, discounts + b * T,
                         values + b * T, (double)bootstrap_values[b], rho_bar, c_bar, clip_eps,
                         cf, T, flip ? flip + b * T : NULL, adv, vt, ratio, surr, pass, rtr, cond, pgw);
        for (int64_t t = 0; t < T; ++t) {
            const double* lpl = lp_th + t * A;
            const double* lpt = lp_tg + t * A;
            double H = 0.0, KL = 0.0;
            for (int64_t k = 0; k < A; ++k) {
                H -= exp(lpl[k]) * lpl[k];
                KL += exp(lpt[k]) * (lpt[k] - lpl[k]);
            }
            double v = (double)values[b * T + t];
            double err = v - vt[t];
            s_surr += surr[t];
            s_val += 0.5 * err * err;
            s_ent += H;
            s_kl += KL;
            s_clip += 1.0 - pass[t];
            s_trunc += rtr[t];
            s_ratio += ratio[t];
            if (dlogits) {
                double* g = dlogits + (b * T + t) * A;
                double w = pgw[t];
                for (int64_t k = 0; k < A; ++k) {
                    double pi = exp(lpl[k]);
                    double onehot = (k == act[t]) ? 1.0 : 0.0;
                    g[k] = (-w * (onehot - pi) + cf->ent_coef * pi * (lpl[k] + H) +
                            cf->kl_coef * (pi - exp(lpt[k]))) / M;
                }
            }
            if (dvalues) dvalues[b * T + t] = cf->vf_coef * err / M;
            if (vtarget_out) vtarget_out[b * T + t] = vt[t];
            if (advantage_out) advantage_out[b * T + t] = adv[t];
            if (ratio_out) ratio_out[b * T + t] = ratio[t];
            if (adv_cond_out) adv_cond_out[b * T + t] = cond[t];
            if (pg_weight_out) pg_weight_out[b * T + t] = pgw[t];
        }
    }
    if (loss_terms) {
        double Lpi = -s_surr / M, LV = s_val / M, H = s_ent / M, KL = s_kl / M;
        loss_terms[0] = Lpi + cf->vf_coef * LV - cf->ent_coef * H + cf->kl_coef * KL;
        loss_terms[1] = Lpi;
        loss_terms[2] = LV;
        loss_terms[3] = H;
        loss_terms[4] = KL;
        loss_terms[5] = s_clip / M;
        loss_terms[6] = s_trunc / M;
        loss_terms[7] = s_ratio / M;
    }
    free(lp_th); free(lp_tg); free(buf);
    return 0;
}

/*
 * Diagonal-Gaussian IMPACT loss (continuous control, Section 4.3; Appendix E assumes a
 * diagonal Gaussian policy).  Per step and dimension d, sigma = exp(logstd):
 *   log pi(a|s)   = sum_d [ -1/2 ((a-mu)/sigma)^2 - logstd - 1/2 ln(2 pi) ]
 *   entropy       = sum_d [ logstd + 1/2 ln(2 pi e) ]
 *   KL(tgt||th)   = sum_d [ logstd_th - logstd_tg + (sigma_tg^2 + (mu_tg-mu_th)^2) / (2 sigma_th^2) - 1/2 ]
 * The rest of the loss is the same as the categorical one.  Gradients are with respect
 * to the learner's mean, log-std and the values.
 */
int oracle_impact_loss_gaussian(
    const float* learner_mean, const float* learner_logstd, const float* target_mean,
    const float* target_logstd, const float* worker_logp, const float* actions,
    const float* rewards, const float* discounts, const float* values,
    const float* bootstrap_values, double rho_bar, double c_bar, double clip_eps,
    const oracle_coef* cf, int64_t B, int64_t T, int64_t D, const int8_t* flip,
    double* loss_terms, double* dmean, double* dlogstd, double* dvalues,
    double* vtarget_out, double* advantage_out, double* ratio_out, double* adv_cond_out,
    double* pg_weight_out) {
    if (B <= 0 || T <= 0 || D <= 0 || !cf) return -1;
    const double M = (double)B * (double)T;
    const double half_log_2pi = 0.5 * log(2.0 * 3.14159265358979323846);
    double* buf = (double*)malloc(sizeof(double) * (size_t)(T * 10));
    if (!buf) return -1;
    double *lth = buf, *ltg = buf + T, *adv = buf + 2 * T, *vt = buf + 3 * T,
           *ratio = buf + 4 * T, *surr = buf + 5 * T, *pass = buf + 6 * T, *rtr = buf + 7 * T,
           *cond = buf + 8 * T, *pgw = buf + 9 * T;
    double s_surr = 0, s_val = 0, s_ent = 0, s_kl = 0, s_clip = 0, s_trunc = 0, s_ratio = 0;

    for (int64_t b = 0; b < B; ++b) {
        for (int64_t t = 0; t < T; ++t) {
            int64_t o = (b * T + t) * D;
            double l1 = 0.0, l2 = 0.0;
            for (int64_t d = 0; d < D; ++d) {
                double a = (double)actions[o + d];
                double z1 = (a - (double)learner_mean[o + d]) / exp((double)learner_logstd[o + d]);
                double z2 = (a - (double)target_mean[o + d]) / exp((double)target_logstd[o + d]);
                l1 += -0.5 * z1 * z1 - (double)learner_logstd[o + d] - half_log_2pi;
                l2 += -0.5 * z2 * z2 - (double)target_logstd[o + d] - half_log_2pi;
            }
            lth[t] = l1;
            ltg[t] = l2;
        }
        trajectory_terms(lth, ltg, worker_logp + b * T, rewards + b * T, discounts + b * T,
                         values + b * T, (double)bootstrap_values[b], rho_bar, c_bar, clip_eps,
                         cf, T, flip ? flip + b * T : NULL, adv, vt, ratio, surr, pass, rtr, cond, pgw);
        for (int64_t t = 0; t < T; ++t) {
            int64_t o = (b * T + t) * D;
            double H = 0.0, KL = 0.0;
            double w = pgw[t];
            for (int64_t d = 0; d < D; ++d) {
                double mu = (double)learner_mean[o + d], ls = (double)learner_logstd[o + d];
                double mut = (double)target_mean[o + d], lst = (double)target_logstd[o + d];
                double var = exp(2.0 * ls), vart = exp(2.0 * lst);
                double a = (double)actions[o + d];
                double dm = mut - mu;
                H += ls + half_log_2pi + 0.5;
                KL += ls - lst + (vart + dm * dm) / (2.0 * var) - 0.5;
                if (dmean) {
                    /* d log pi / d mu = (a - mu) / sigma^2 ;  d KL / d mu = (mu - mu_tg) / sigma^2 */
                    dmean[o + d] = (-w * (a - mu) / var + cf->kl_coef * (mu - mut) / var) / M;
                }
                if (dlogstd) {
                    /* d log pi / d logstd = ((a-mu)/sigma)^2 - 1 ; d H / d logstd = 1 ;
                       d KL / d logstd = 1 - (sigma_tg^2 + (mu_tg-mu)^2) / sigma^2 */
                    double z = (a - mu) * (a - mu) / var;
                    dlogstd[o + d] = (-w * (z - 1.0) - cf->ent_coef +
                                      cf->kl_coef * (1.0 - (vart + dm * dm) / var)) / M;
                }
            }
            double v = (double)values[b * T + t];
            double err = v - vt[t];
            s_surr += surr[t];
            s_val += 0.5 * err * err;
            s_ent += H;
            s_kl += KL;
            s_clip += 1.0 - pass[t];
            s_trunc += rtr[t];
            s_ratio += ratio[t];
            if (dvalues) dvalues[b * T + t] = cf->vf_coef * err / M;
            if (vtarget_out) vtarget_out[b * T + t] = vt[t];
            if (advantage_out) advantage_out[b * T + t] = adv[t];
            if (ratio_out) ratio_out[b * T + t] = ratio[t];
            if (adv_cond_out) adv_cond_out[b * T + t] = cond[t];
            if (pg_weight_out) pg_weight_out[b * T + t] = pgw[t];
        }
    }
    if (loss_terms) {
        double Lpi = -s_surr / M, LV = s_val / M, H = s_ent / M, KL = s_kl / M;
        loss_terms[0] = Lpi + cf->vf_coef * LV - cf->ent_coef * H + cf->kl_coef * KL;
        loss_terms[1] = Lpi;
        loss_terms[2] = LV;
        loss_terms[3] = H;
        loss_terms[4] = KL;
        loss_terms[5] = s_clip / M;
        loss_terms[6] = s_trunc / M;
        loss_terms[7] = s_ratio / M;
    }
    free(buf);
    return 0;
}

/* ------------------------------------------------------------------------------------
 * Circular buffer C(N, K) (Algorithm 1; Section 3.2): N batches, each handed to the
 * learner at most K times, then discarded and replaced by a new worker batch.
 * Metadata only; the payload of a slot is the caller's business (tests keep it in NumPy).
 * ------------------------------------------------------------------------------------ */

#define ORING_OK 0
#define ORING_EMPTY 1
#define ORING_FULL 2

typedef struct {
    int32_t N, K, mode;     /* mode 0: uniform draw over live slots, 1: round robin */
    int32_t write_cursor, read_cursor;
    uint64_t seed, draws;
    int32_t* valid;
    int32_t* count;
} oracle_ring;

/* n-th output of the SplitMix64 generator started at `seed` (Steele, Lea, Flood 2014):
 * a counter-based draw, so the sequence is a pure function of (seed, n). */
static uint64_t draw_u64(uint64_t seed, uint64_t n) {
    uint64_t z = seed + (n + 1u) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

oracle_ring* oracle_ring_create(int32_t N, int32_t K, int32_t mode, uint64_t seed) {
    if (N <= 0 || K <= 0 || (mode != 0 && mode != 1)) return NULL;
    oracle_ring* r = (oracle_ring*)calloc(1, sizeof(oracle_ring));
    r->N = N; r->K = K; r->mode = mode; r->seed = seed;
    r->valid = (int32_t*)calloc((size_t)N, sizeof(int32_t));
    r->count = (int32_t*)calloc((size_t)N, sizeof(int32_t));
    return r;
}

void oracle_ring_destroy(oracle_ring* r) {
    if (!r) return;
    free(r->valid); free(r->count); free(r);
}

/* A worker batch goes to the first free slot at or after the write cursor, in ring
 * order; with every slot still live the buffer is full and nothing changes. */
int32_t oracle_ring_push(oracle_ring* r, int32_t* slot_out) {
    for (int32_t i = 0; i < r->N; ++i) {
        int32_t s = (r->write_cursor + i) % r->N;
        if (!r->valid[s]) {
            r->valid[s] = 1;
            r->count[s] = 0;
            r->write_cursor = (s + 1) % r->N;
            *slot_out = s;
            return ORING_OK;
        }
    }
    return ORING_FULL;
}

/* The learner obtains a batch that has been traversed k times (k returned before the
 * increment); after its K-th traversal the batch is discarded. */
int32_t oracle_ring_sample(oracle_ring* r, int32_t* slot_out, int32_t* k_out) {
    int32_t live = 0;
    for (int32_t s = 0; s < r->N; ++s) live += r->valid[s] ? 1 : 0;
    if (live == 0) return ORING_EMPTY;
    int32_t pick = -1;
    if (r->mode == 0) {
        uint64_t u = draw_u64(r->seed, r->draws++);
        /* floor(u * live / 2^64) without modulo bias */
        uint64_t j = (uint64_t)(((unsigned __int128)u * (unsigned __int128)(uint64_t)live) >> 64);
        for (int32_t s = 0; s < r->N; ++s) {
            if (r->valid[s]) {
                if (j == 0) { pick = s; break; }
                --j;
            }
        }
    } else {
        for (int32_t i = 0; i < r->N; ++i) {
            int32_t s = (r->read_cursor + i) % r->N;
            if (r->valid[s]) { pick = s; break; }
        }
        r->read_cursor = (pick + 1) % r->N;
    }
    *slot_out = pick;
    *k_out = r->count[pick];
    r->count[pick] += 1;
    if (r->count[pick] >= r->K) r->valid[pick] = 0;
    return ORING_OK;
}

int32_t oracle_ring_live(const oracle_ring* r) {
    int32_t live = 0;
    for (int32_t s = 0; s < r->N; ++s) live += r->valid[s] ? 1 : 0;
    return live;
}

uint64_t oracle_draw_u64(uint64_t seed, uint64_t n) { return draw_u64(seed, n); }
