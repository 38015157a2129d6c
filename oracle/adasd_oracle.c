/*
 * AdaSD oracle: a plain, slow, float64 CPU statement of what the hot path computes.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may call, link or import
 * this file; it shares no code with the CUDA library.  It exists so that the CUDA
 * kernels can be checked element by element against the paper's definitions.
 *
 * Every function cites the passage of the paper it follows.  There is no blocking,
 * fusion or reordering: sums run left to right in index order.
 *
 * Pins (tests marked "not gpu"): closed forms H(uniform)=ln V, H(one-hot)=0,
 * JSD(p,p)=0, symmetry, JSD<=ln 2 with equality on disjoint supports (distance exactly
 * 1 there, exactly 0 on coinciding rows, whatever the rounding of the sum), equality of
 * the two printed forms of the JS divergence, KL = CE - H, triangle inequality of
 * the JS distance, hand-derived V=4 values, brute-force inverse CDF, Leviathan's
 * output-law identity for the vanilla mode, KDE against quadrature and library
 * routines, running-mean threshold trajectories; the adjusted distribution (temperature,
 * top-k, top-p) against a hand-derived V=8 row, p^(1/T), a partition, an independent
 * sort-and-cumsum rule and its minimality.
 *
 * Parity unpinned (the paper does not fix them; the readings are listed in the
 * design notes): the KDE kernel and bandwidth rule, the cold-start rule for the
 * Bayes posterior, and the meaning of Reject(P(A|d)).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_BF16 0
#define ORACLE_FP32 1
#define ORACLE_F64 2   /* rows already in double: the output of oracle_warp_logits */

static size_t elt_size(int32_t dtype) { return dtype == ORACLE_BF16 ? 2 : dtype == ORACLE_FP32 ? 4 : 8; }

/* ---------------------------------------------------------------- input widening */

/* Logits exactly as the device receives them (bf16 bits or fp32), widened to double. */
void oracle_widen(const void* z, int32_t dtype, int64_t n, double* out) {
    if (dtype == ORACLE_BF16) {
        const uint16_t* h = (const uint16_t*)z;
        for (int64_t i = 0; i < n; ++i) {
            union { uint32_t u; float f; } c;
            c.u = (uint32_t)h[i] << 16;
            out[i] = (double)c.f;
        }
    } else if (dtype == ORACLE_FP32) {
        const float* f = (const float*)z;
        for (int64_t i = 0; i < n; ++i) out[i] = (double)f[i];
    } else {
        memcpy(out, z, sizeof(double) * (size_t)n);
    }
}

/* ---------------------------------------------------------------- per-row definitions */

/*
 * Softmax of a logit row (Sec. 2.1.1: the model's probability distribution over the
 * vocabulary).  Returns the log-sum-exp; p sums to 1.  -inf logits get p = 0.
 * A row with no finite logit, or with a NaN, yields NaN everywhere.
 */
double oracle_softmax(const double* z, int32_t V, double* p) {
    double m = -INFINITY;
    int bad = 0;
    for (int32_t v = 0; v < V; ++v) {
        if (isnan(z[v])) bad = 1;
        if (z[v] > m) m = z[v];
    }
    if (bad || !isfinite(m)) {
        for (int32_t v = 0; v < V; ++v) p[v] = NAN;
        return NAN;
    }
    double S = 0.0;
    for (int32_t v = 0; v < V; ++v) {
        p[v] = exp(z[v] - m);
        S += p[v];
    }
    for (int32_t v = 0; v < V; ++v) p[v] /= S;
    return m + log(S);
}

/* Entropy H(p) = -sum p log p in nats, 0 log 0 := 0 (Appendix A, entropy).
 * NaN for the NaN row that oracle_softmax gives an unusable logit row. */
double oracle_entropy(const double* p, int32_t V) {
    double H = 0.0;
    for (int32_t v = 0; v < V; ++v) {
        if (isnan(p[v])) return NAN;
        if (p[v] > 0.0) H -= p[v] * log(p[v]);
    }
    return H;
}

/* Cross-entropy H(p,q) = -sum p log q (Appendix A). +inf where p>0 and q=0. */
double oracle_cross_entropy(const double* p, const double* q, int32_t V) {
    double H = 0.0;
    for (int32_t v = 0; v < V; ++v)
        if (p[v] > 0.0) H -= p[v] * log(q[v]);
    return H;
}

/* KL divergence sum p log(p/q) (Appendix A). */
double oracle_kl(const double* p, const double* q, int32_t V) {
    double D = 0.0;
    for (int32_t v = 0; v < V; ++v)
        if (p[v] > 0.0) D += p[v] * log(p[v] / q[v]);
    return D;
}

/*
 * JS divergence, first printed form (Sec. 2.2):
 *   D_JS(p||q) = 1/2 KL(p||m) + 1/2 KL(q||m),  m = (p+q)/2,   in nats.
 * Terms with a zero numerator are dropped.  p is the target row, q the draft row.
 */
double oracle_jsd(const double* p, const double* q, int32_t V) {
    double D = 0.0;
    for (int32_t v = 0; v < V; ++v) {
        double mv = 0.5 * (p[v] + q[v]);
        double t = 0.0;
        if (p[v] > 0.0) t += p[v] * log(p[v] / mv);
        if (q[v] > 0.0) t += q[v] * log(q[v] / mv);
        D += 0.5 * t;
    }
    return D;
}

/* JS divergence, second printed form (Sec. 2.2): H(m) - (H(p)+H(q))/2. */
double oracle_jsd_entropy_form(const double* p, const double* q, int32_t V) {
    double Hm = 0.0;
    for (int32_t v = 0; v < V; ++v) {
        double mv = 0.5 * (p[v] + q[v]);
        if (mv > 0.0) Hm -= mv * log(mv);
    }
    return Hm - 0.5 * (oracle_entropy(p, V) + oracle_entropy(q, V));
}

/*
 * JS distance d_JS = sqrt(D_JS) (Sec. 2.2), with the divergence taken in base 2 so
 * that d lies in [0,1] and "exactly 0 or 1" (Sec. 4.4) means what it says:
 * d = sqrt(clamp(D_JS_nats, 0, ln 2) / ln 2).
 */
double oracle_js_distance(double jsd_nats) {
    const double ln2 = 0.69314718055994530942;
    double c = jsd_nats;
    if (isnan(c)) return NAN;
    if (c < 0.0) c = 0.0;
    if (c > ln2) c = ln2;
    return sqrt(c / ln2);
}

/*
 * The two ends of the distance (Sec. 4.4: samples whose distance is exactly 0 or 1 stay
 * out of the KDE lists; the paper meets them where the two distributions coincide or
 * share no token, as truncated sampling distributions do).  A sum of V rounded terms
 * cannot be relied on to land on 0 or ln 2 to the last bit, so the ends are decided by
 * what defines them: p_v = q_v for every v gives D_JS = 0 and d = 0; no v with p_v > 0
 * and q_v > 0 (disjoint supports) gives D_JS = ln 2 and d = 1.  Every other pair takes
 * the sum of oracle_jsd and the clamp of oracle_js_distance (which may itself round to
 * an end).  Returns d and stores D_JS in nats.
 */
double oracle_js_distance_rows(const double* p, const double* q, int32_t V, double* jsd_out) {
    const double ln2 = 0.69314718055994530942;
    int identical = 1, disjoint = 1;
    for (int32_t v = 0; v < V; ++v) {
        if (isnan(p[v]) || isnan(q[v])) {
            *jsd_out = NAN;
            return NAN;
        }
        if (p[v] != q[v]) identical = 0;
        if (p[v] > 0.0 && q[v] > 0.0) disjoint = 0;
    }
    if (identical) {
        *jsd_out = 0.0;
        return 0.0;
    }
    if (disjoint) {
        *jsd_out = ln2;
        return 1.0;
    }
    *jsd_out = oracle_jsd(p, q, V);
    return oracle_js_distance(*jsd_out);
}

/*
 * Inverse-CDF sample (Alg. 1 "x_i ~ q_i", "y_i ~ p_i") with a caller-supplied
 * uniform u in [0,1): the smallest v with C_v = sum_{j<=v} p_j > u, scanning in
 * index order; if rounding leaves none, the largest v with p_v > 0.  margin_out
 * receives min(u - C_{v-1}, C_v - u): how far u is from the nearest CDF edge.
 */
int32_t oracle_inv_cdf(const double* p, int32_t V, double u, double* margin_out) {
    double C = 0.0;
    int32_t last_pos = -1;
    for (int32_t v = 0; v < V; ++v) {
        double prev = C;
        if (p[v] > 0.0) last_pos = v;
        C += p[v];
        if (C > u) {
            if (margin_out) {
                double a = u - prev, b = C - u;
                *margin_out = a < b ? a : b;
            }
            return v;
        }
    }
    if (margin_out) *margin_out = 0.0;
    return last_pos;
}

/* ---------------------------------------------------------------- adjusted distribution */

typedef struct { double z; int32_t v; } warp_item;
static int warp_desc(const void* a, const void* b) {
    const warp_item* x = (const warp_item*)a;
    const warp_item* y = (const warp_item*)b;
    if (x->z > y->z) return -1;
    if (x->z < y->z) return 1;
    return (x->v > y->v) - (x->v < y->v);
}

/*
 * The adjusted distribution a token is sampled from (Sec. 2.1.1: temperature scaling,
 * top-k sampling, top-p sampling), as logits: out_v = z_v / temperature for the tokens
 * that stay, -inf for the tokens that are cut, applied in that order.
 *
 *   temperature > 0        z_v / temperature.
 *   0 < top_k < V          the k most probable tokens stay; tokens whose logit equals the
 *                          k-th largest stay with it (a tie is never split).
 *   0 < top_p < 1          with pi = softmax of what the first two steps left, a token
 *                          stays iff the tokens STRICTLY more probable than it hold less
 *                          than top_p of the mass: the smallest set of most probable
 *                          tokens whose mass reaches top_p, ties at its edge included.
 *   top_k <= 0 or >= V, top_p >= 1, temperature == 1: that step changes nothing.
 *
 * margin_out: the smallest |mass of the strictly more probable tokens - top_p| over the
 * groups of equally probable tokens, i.e. how close the top-p decision came to going the
 * other way (+inf when top-p is off).  band_mass_out: the mass of the groups whose decision
 * lies within `band` of going the other way (what a checker that sums the same masses in
 * lower precision may decide differently).  A row with NaN or without a finite logit is
 * returned scaled and uncut.
 */
void oracle_warp_logits(const double* z, int32_t V, double temperature, int32_t top_k, double top_p,
                        double band, double* out, double* margin_out, double* band_mass_out) {
    *margin_out = INFINITY;
    *band_mass_out = 0.0;
    int bad = 0, finite = 0;
    for (int32_t v = 0; v < V; ++v) {
        out[v] = z[v] / temperature;
        if (isnan(z[v])) bad = 1;
        if (isfinite(z[v])) finite = 1;
        if (z[v] == INFINITY) bad = 1;
    }
    if (bad || !finite) return;
    warp_item* it = (warp_item*)malloc(sizeof(warp_item) * (size_t)V);
    if (top_k > 0 && top_k < V) {
        for (int32_t v = 0; v < V; ++v) { it[v].z = out[v]; it[v].v = v; }
        qsort(it, (size_t)V, sizeof(warp_item), warp_desc);
        const double kth = it[top_k - 1].z;
        for (int32_t v = 0; v < V; ++v)
            if (out[v] < kth) out[v] = -INFINITY;
    }
    if (top_p > 0.0 && top_p < 1.0) {
        double* pi = (double*)malloc(sizeof(double) * (size_t)V);
        oracle_softmax(out, V, pi);
        for (int32_t v = 0; v < V; ++v) { it[v].z = out[v]; it[v].v = v; }
        qsort(it, (size_t)V, sizeof(warp_item), warp_desc);
        double above = 0.0;                 /* mass of the tokens strictly more probable than the group */
        int32_t s = 0;
        while (s < V && it[s].z > -INFINITY) {
            int32_t e = s;
            double group = 0.0;
            while (e < V && it[e].z == it[s].z) { group += pi[it[e].v]; ++e; }
            const double gap = fabs(above - top_p);
            if (gap < *margin_out) *margin_out = gap;
            if (gap < band) *band_mass_out += group;
            if (!(above < top_p))
                for (int32_t i = s; i < e; ++i) out[it[i].v] = -INFINITY;
            above += group;
            s = e;
        }
        free(pi);
    }
    free(it);
}

/* ---------------------------------------------------------------- KDE and Bayes (Sec. 4.4) */

/* sample standard deviation (n-1 in the denominator); 0 for n<2 */
double oracle_sample_std(const double* x, int32_t n) {
    if (n < 2) return 0.0;
    double mean = 0.0;
    for (int32_t i = 0; i < n; ++i) mean += x[i];
    mean /= (double)n;
    double ss = 0.0;
    for (int32_t i = 0; i < n; ++i) ss += (x[i] - mean) * (x[i] - mean);
    return sqrt(ss / (double)(n - 1));
}

/* bandwidth h = std * factor(n); rule 0: Silverman (3n/4)^(-1/5), rule 1: Scott n^(-1/5) */
double oracle_kde_bandwidth(const double* x, int32_t n, int32_t rule) {
    double sd = oracle_sample_std(x, n);
    double f = rule == 0 ? pow(0.75 * (double)n, -0.2) : pow((double)n, -0.2);
    return sd * f;
}

/*
 * Gaussian kernel density estimate at x over the list (Sec. 4.4, "KDE(L, d)"):
 *   f(x) = 1/(n h sqrt(2 pi)) sum_j exp(-(x - x_j)^2 / (2 h^2)).
 */
double oracle_kde(const double* list, int32_t n, double x, int32_t rule) {
    double h = oracle_kde_bandwidth(list, n, rule);
    if (n < 1 || !(h > 0.0)) return NAN;
    double acc = 0.0;
    for (int32_t j = 0; j < n; ++j) {
        double t = (x - list[j]) / h;
        acc += exp(-0.5 * t * t);
    }
    return acc / ((double)n * h * 2.50662827463100050242);
}

/*
 * Bayesian acceptance probability (Sec. 4.4; Alg. 1, the posterior lines):
 *   P(A|d) = p(d|A) P(A) / (p(d|A) P(A) + p(d|R) P(R)),  P(A) = |L_A|/(|L_A|+|L_R|).
 * Cold start (reading): if either list has fewer than min_samples entries, either
 * sample deviation is 0, or the denominator is 0 or not finite, P(A|d) := 0, i.e.
 * verification falls back to exact token match.
 */
double oracle_accept_prob(const double* LA, int32_t nA, const double* LR, int32_t nR, double d,
                          int32_t min_samples, int32_t rule) {
    if (nA < min_samples || nR < min_samples || nA < 2 || nR < 2) return 0.0;
    double fA = oracle_kde(LA, nA, d, rule);
    double fR = oracle_kde(LR, nR, d, rule);
    if (isnan(fA) || isnan(fR)) return 0.0;
    double PA = (double)nA / (double)(nA + nR);
    double PR = (double)nR / (double)(nA + nR);
    double num = fA * PA;
    double den = fA * PA + fR * PR;
    if (!(den > 0.0) || !isfinite(den)) return 0.0;
    return num / den;
}

/* ---------------------------------------------------------------- draft step (Sec. 4.3) */

/*
 * One draft step for one sequence (Alg. 1, generation loop body): softmax of the
 * draft row, H(q_i), x_i ~ q_i by inverse CDF with uniform u, and the stop check
 * H(q_i) > T_G (strict).  The token that trips the check stays in the window; the
 * caller counts it.
 */
void oracle_draft_step(const void* z, int32_t dtype, int32_t V, double u, double T_G,
                       double* H_out, double* lse_out, int32_t* token_out, double* margin_out,
                       int32_t* stop_out) {
    double* zz = (double*)malloc(sizeof(double) * (size_t)V);
    double* p = (double*)malloc(sizeof(double) * (size_t)V);
    oracle_widen(z, dtype, V, zz);
    double lse = oracle_softmax(zz, V, p);
    double H = oracle_entropy(p, V);
    *H_out = H;
    *lse_out = lse;
    *token_out = isnan(lse) ? -1 : oracle_inv_cdf(p, V, u, margin_out);
    *stop_out = (H > T_G) ? 1 : 0;
    free(zz);
    free(p);
}

/* ---------------------------------------------------------------- per-position math */

/*
 * Definitions evaluated at every candidate position of one sequence: softmax of the
 * draft row q_i and target row p_i, their entropies, D_JS(p_i||q_i), d_i, and the
 * target sample y_i ~ p_i (Alg. 1, "y_1..y_{w+1} ~ p_1..p_{w+1}").  Row K_t of the
 * target (the bonus row) has no draft partner.  Rows are independent, so positions
 * run in parallel.
 */
static void position_math(const void* zd, const void* zt, int32_t dtype, int32_t V,
                          int64_t d_row_stride, int64_t t_row_stride, int32_t K_t,
                          const float* u_target, double* H_d, double* H_t, double* lse_d,
                          double* lse_t, double* jsd, double* dist, int32_t* y,
                          double* y_margin) {
    size_t esz = elt_size(dtype);
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t i = 0; i <= K_t; ++i) {
        double* zz = (double*)malloc(sizeof(double) * (size_t)V);
        double* p = (double*)malloc(sizeof(double) * (size_t)V);
        double* q = (double*)malloc(sizeof(double) * (size_t)V);
        oracle_widen((const char*)zt + (size_t)i * (size_t)t_row_stride * esz, dtype, V, zz);
        lse_t[i] = oracle_softmax(zz, V, p);
        H_t[i] = oracle_entropy(p, V);
        double mg = 0.0;
        y[i] = isnan(lse_t[i]) ? -1 : oracle_inv_cdf(p, V, (double)u_target[i], &mg);
        y_margin[i] = mg;
        if (i < K_t) {
            oracle_widen((const char*)zd + (size_t)i * (size_t)d_row_stride * esz, dtype, V, zz);
            lse_d[i] = oracle_softmax(zz, V, q);
            H_d[i] = oracle_entropy(q, V);
            dist[i] = oracle_js_distance_rows(p, q, V, &jsd[i]);
        }
        free(zz);
        free(p);
        free(q);
    }
}

/* ---------------------------------------------------------------- AdaSD round (Alg. 1) */

/*
 * Verification and update of one round for one sequence, in the listing's order.
 *
 * In:  K_t draft rows and K_t+1 target rows, draft tokens x[K_t], uniforms
 *      u_target[K_t+1] (for y_i) and u_accept[K_t] (for the accept draw), the lists
 *      L_E^R (LE,nE), L_D^A (LA,nA), L_D^R (LR,nR) with room for this round's appends,
 *      and T_G.
 * Out: per-position H_d, H_t, lse_d, lse_t, jsd, dist, y, y_margin (all positions);
 *      p_acc[i] = P(A|d_i) for the positions the loop reached (NaN beyond the break);
 *      accept_len, next_token = y[accept_len], rejected (1 if the loop broke).
 *
 * reject_rule 0: Reject(P) is a Bernoulli draw, reject iff u_accept[i] >= P(A|d_i);
 * reject_rule 1: reject iff P(A|d_i) < 1/2.  A match x_i = y_i always accepts.
 */
void oracle_verify_round(const void* zd, const void* zt, int32_t dtype, int32_t V,
                         int64_t d_row_stride, int64_t t_row_stride, int32_t K_t,
                         const int32_t* x, const float* u_target, const float* u_accept,
                         double* LE, int32_t* nE, double* LA, int32_t* nA, double* LR,
                         int32_t* nR, double* T_G, int32_t min_samples, int32_t bw_rule,
                         int32_t reject_rule, int32_t update, double* H_d, double* H_t,
                         double* lse_d, double* lse_t, double* jsd, double* dist, double* p_acc,
                         int32_t* y, double* y_margin, int32_t* accept_len, int32_t* next_token,
                         int32_t* rejected) {
    position_math(zd, zt, dtype, V, d_row_stride, t_row_stride, K_t, u_target, H_d, H_t, lse_d,
                  lse_t, jsd, dist, y, y_margin);
    for (int32_t i = 0; i < K_t; ++i) p_acc[i] = NAN;

    /* when update == 0 the lists must come out unchanged: work on private copies */
    int32_t nE0 = *nE, nA0 = *nA, nR0 = *nR;
    double* LAw = LA;
    if (!update) {
        LAw = (double*)malloc(sizeof(double) * (size_t)(nA0 + K_t + 1));
        memcpy(LAw, LA, sizeof(double) * (size_t)nA0);
    }
    int32_t nAw = nA0, nRw = nR0, nEw = nE0;

    int32_t w = K_t;
    int32_t broke = 0;
    for (int32_t i = 0; i < K_t; ++i) {              /* i is the listing's i-1 */
        double d = dist[i];
        double PA = oracle_accept_prob(LAw, nAw, LR, nRw, d, min_samples, bw_rule);
        p_acc[i] = PA;
        int rej = reject_rule == 0 ? ((double)u_accept[i] >= PA) : (PA < 0.5);
        if (x[i] != y[i] && rej) {
            /* record rejected entropy; a position one of whose rows holds NaN or no finite
             * logit has no distance, and nothing of it is recorded (the paper is silent on
             * such rows: they are rejected and leave the lists, and so T_G, as they were) */
            if (isfinite(H_d[i]) && !isnan(d)) {
                if (update) LE[nEw] = H_d[i];
                nEw++;
            }
            if (update && 0.0 < d && d < 1.0) LR[nRw++] = d;
            w = i;                                    /* w <- i - 1 in 1-based terms */
            broke = 1;
            break;
        }
        if (0.0 < d && d < 1.0) LAw[nAw++] = d;       /* record accepted distance */
    }
    *accept_len = w;
    *next_token = y[w];
    *rejected = broke;
    if (update) {
        *nE = nEw;
        *nA = nAw;
        *nR = nRw;
        if (nEw > 0) {                                /* T_G <- average(L_E^R) */
            double s = 0.0;
            for (int32_t j = 0; j < nEw; ++j) s += LE[j];
            *T_G = s / (double)nEw;
        }
    } else {
        free(LAw);
    }
}

/* ---------------------------------------------------------------- vanilla round (Sec. 2.1.3) */

/*
 * Vanilla speculative sampling for one sequence: for i = 1..K accept x_i iff
 * u_accept[i] < alpha_i = min(1, p_i(x_i)/q_i(x_i)); at the first rejection the next
 * token is drawn from norm(max(0, p_i - q_i)) with uniform u_resample (from p_i if
 * that residual has no mass); if nothing is rejected the next token is drawn from
 * the bonus row p_{K+1} with u_resample.
 */
void oracle_vanilla_round(const void* zd, const void* zt, int32_t dtype, int32_t V,
                          int64_t d_row_stride, int64_t t_row_stride, int32_t K,
                          const int32_t* x, const float* u_accept, double u_resample,
                          double* alpha, int32_t* accept_len, int32_t* next_token,
                          double* resample_margin) {
    size_t esz = elt_size(dtype);
    double* zz = (double*)malloc(sizeof(double) * (size_t)V);
    double* p = (double*)malloc(sizeof(double) * (size_t)V);
    double* q = (double*)malloc(sizeof(double) * (size_t)V);
    int32_t w = K;
    for (int32_t i = 0; i < K; ++i) alpha[i] = NAN;
    *resample_margin = 0.0;
    for (int32_t i = 0; i < K; ++i) {
        oracle_widen((const char*)zt + (size_t)i * (size_t)t_row_stride * esz, dtype, V, zz);
        oracle_softmax(zz, V, p);
        oracle_widen((const char*)zd + (size_t)i * (size_t)d_row_stride * esz, dtype, V, zz);
        oracle_softmax(zz, V, q);
        double a = p[x[i]] / q[x[i]];
        if (a > 1.0) a = 1.0;
        alpha[i] = a;
        if (!((double)u_accept[i] < a)) {
            double R = 0.0;
            for (int32_t v = 0; v < V; ++v) {
                double r = p[v] - q[v];
                zz[v] = r > 0.0 ? r : 0.0;
                R += zz[v];
            }
            if (R > 0.0) {
                for (int32_t v = 0; v < V; ++v) zz[v] /= R;
                *next_token = oracle_inv_cdf(zz, V, u_resample, resample_margin);
            } else {
                *next_token = oracle_inv_cdf(p, V, u_resample, resample_margin);
            }
            w = i;
            break;
        }
    }
    if (w == K) {
        oracle_widen((const char*)zt + (size_t)K * (size_t)t_row_stride * esz, dtype, V, zz);
        oracle_softmax(zz, V, p);
        *next_token = oracle_inv_cdf(p, V, u_resample, resample_margin);
    }
    *accept_len = w;
    free(zz);
    free(p);
    free(q);
}

/* ---------------------------------------------------------------- greedy decoding (Sec. 2.1.3) */

/*
 * The most probable token of a logit row, x = argmax_v z_v (Sec. 2.1.1, deterministic
 * selection); among equal maxima the lowest index.  -1 for a row with NaN or without a
 * finite logit.
 */
int32_t oracle_argmax(const void* z, int32_t dtype, int32_t V) {
    double* zz = (double*)malloc(sizeof(double) * (size_t)V);
    oracle_widen(z, dtype, V, zz);
    int32_t best = -1;
    double m = -INFINITY;
    int bad = 0;
    for (int32_t v = 0; v < V; ++v) {
        if (isnan(zz[v])) bad = 1;
        if (zz[v] > m) {
            m = zz[v];
            best = v;
        }
    }
    free(zz);
    return (bad || !isfinite(m)) ? -1 : best;
}

/*
 * Greedy verification of one round for one sequence (Sec. 2.1.3, greedy decoding): the
 * candidate x_i is accepted only if it equals the target's own choice argmax p_i; the scan
 * stops at the first mismatch, and the token emitted after the accepted prefix is the
 * target's choice at that position (the bonus row's if every candidate matched).
 * argmax_out[K+1] receives the target's choices of the rows the scan looked at (-2 beyond).
 */
void oracle_greedy_round(const void* zt, int32_t dtype, int32_t V, int64_t t_row_stride, int32_t K,
                         const int32_t* x, int32_t* argmax_out, int32_t* accept_len,
                         int32_t* next_token) {
    size_t esz = elt_size(dtype);
    int32_t w = K;
    for (int32_t i = 0; i <= K; ++i) argmax_out[i] = -2;
    for (int32_t i = 0; i < K; ++i) {
        argmax_out[i] = oracle_argmax((const char*)zt + (size_t)i * (size_t)t_row_stride * esz, dtype, V);
        if (x[i] != argmax_out[i]) {
            w = i;
            break;
        }
    }
    if (w == K)
        argmax_out[K] = oracle_argmax((const char*)zt + (size_t)K * (size_t)t_row_stride * esz, dtype, V);
    *accept_len = w;
    *next_token = argmax_out[w];
}

/* ---------------------------------------------------------------- ablation variants (Sec. 5) */

/*
 * Gen-Only (Sec. 5, ablation): the generation component alone.  The draft loop stops on
 * H(q_i) > T_G as in Alg. 1, verification is vanilla speculative sampling, and the feedback
 * that T_G needs is the entropy of the rejected candidate: if vanilla verification rejected
 * candidate accept_len (accept_len < K_t), H(q_{accept_len}) joins L_E^R and T_G becomes the
 * mean of the list (Sec. 4.3).  No distances are collected.  H_d[K_t] are the entropies the
 * draft steps produced.  (Verify-Only needs no function of its own: it is oracle_verify_round
 * on a fixed window of five candidates.)
 */
void oracle_gen_only_update(double* LE, int32_t* nE, double* T_G, const double* H_d, int32_t K_t,
                            int32_t accept_len) {
    if (accept_len < 0 || accept_len >= K_t) return;          /* nothing was rejected */
    if (!isfinite(H_d[accept_len])) return;
    LE[*nE] = H_d[accept_len];
    *nE += 1;
    double s = 0.0;
    for (int32_t j = 0; j < *nE; ++j) s += LE[j];
    *T_G = s / (double)*nE;
}
