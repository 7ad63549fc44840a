/*
 * Power-SMC CPU oracle -- TEST INFRASTRUCTURE ONLY (see psmc_oracle.h).
 *
 * Double precision, sequential sums in index order, the steps of Algorithm 1
 * in the order the paper lists them.  OpenMP is used only across rows of one
 * step (rows are independent in Algorithm 1's inner loop); every per-row and
 * per-group computation is a plain sequential loop.
 */
#include "psmc_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ */
/* randomness: splitmix64 finaliser chained over a 5-part counter      */
/* ------------------------------------------------------------------ */
uint64_t orc_sm64(uint64_t x) {
    uint64_t z = x + 0x9E3779B97F4A7C15ULL;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

uint64_t orc_hash5(uint64_t a, uint64_t b, uint64_t c, uint64_t d, uint64_t e) {
    uint64_t h = orc_sm64(a);
    h = orc_sm64(h ^ b);
    h = orc_sm64(h ^ c);
    h = orc_sm64(h ^ d);
    h = orc_sm64(h ^ e);
    return h;
}

/* top 52 bits, centred: every step below is exact in double, so U lies strictly inside (0,1) */
double orc_uniform(uint64_t h) { return ((double)(h >> 12) + 0.5) * (1.0 / 4503599627370496.0); }

/* ------------------------------------------------------------------ */
/* exponent schedule, Section 4.3: one stage per token, linear in t    */
/* ------------------------------------------------------------------ */
double orc_alpha_at(double alpha, int ramp, int t) {
    if (ramp <= 0) return alpha; /* no bridging: the target exponent from the start */
    int s = t < ramp ? t : ramp;
    return 1.0 + (alpha - 1.0) * (double)s / (double)ramp;
}

double orc_beta_at(double alpha, double tau, int ramp, int t) {
    return orc_alpha_at(alpha, ramp, t) / (alpha * tau);
}

/* ------------------------------------------------------------------ */
/* one row                                                             */
/* ------------------------------------------------------------------ */
int orc_row(const double* l, int V, double beta, double alpha_t, double U, int force, int* y,
            int* y_own, double* logp_y, double* logq_y, double* log_omega, double* L1,
            double* Lbeta, double* margin) {
    double m = -INFINITY;
    for (int v = 0; v < V; ++v) {
        if (isnan(l[v]) || l[v] == INFINITY) return 5;
        if (l[v] > m) m = l[v];
    }
    if (m == -INFINITY) return 5;

    /* log-softmax normaliser of p = softmax(l) */
    double sum1 = 0.0;
    for (int v = 0; v < V; ++v) sum1 += exp(l[v] - m);
    double l1 = m + log(sum1);

    /* proposal q = softmax(beta * l) (Corollary 1: temperature 1/beta) */
    double total = 0.0;
    for (int v = 0; v < V; ++v) total += exp(beta * (l[v] - m));
    double lb = beta * m + log(total);

    /* inverse CDF in vocabulary order: first v whose inclusive prefix reaches U * total */
    double target = U * total;
    double cum = 0.0, below = 0.0, at = 0.0;
    int pick = -1, last_pos = -1;
    for (int v = 0; v < V; ++v) {
        double e = exp(beta * (l[v] - m));
        double prev = cum;
        cum += e;
        if (e > 0.0) last_pos = v;
        if (pick < 0 && cum >= target) {
            pick = v;
            below = prev;
            at = cum;
        }
    }
    if (pick < 0) { /* rounding left the last prefix short of the target */
        pick = last_pos;
        below = at = total;
    }
    double mg = 1.0;
    if (below > 0.0) mg = fmin(mg, fabs(U - below / total));
    /* the upper fence exists whenever a later token has mass, even one too small to move the fp64 prefix */
    if (pick < last_pos) mg = fmin(mg, fabs(at / total - U));

    int tok = force >= 0 ? force : pick;
    double lp = l[tok] - l1;
    double lq = beta * l[tok] - lb;
    *y = tok;
    *y_own = pick;
    *logp_y = lp;
    *logq_y = lq;
    *log_omega = alpha_t * lp - lq; /* Eq. 7 in logs */
    *L1 = l1;
    *Lbeta = lb;
    *margin = mg;
    return 0;
}

/* ------------------------------------------------------------------ */
/* one row, proposal restricted to the top of the row                  */
/* ------------------------------------------------------------------ */
typedef struct { double l; int v; } ranked_t;
static int by_logit_then_id(const void* a, const void* b) {
    const ranked_t* x = (const ranked_t*)a;
    const ranked_t* y = (const ranked_t*)b;
    if (x->l > y->l) return -1;
    if (x->l < y->l) return 1;
    return (x->v > y->v) - (x->v < y->v);
}

int orc_row_masked(const double* l, int V, double beta, double alpha_t, double U, int top_k, double top_p,
                   int force_k, int force_tok, int* y, int* y_own, int* k_used, int* k_own, double* k_margin,
                   double* logp_y, double* logq_y, double* log_omega, double* margin) {
    if ((top_k > 0) == (top_p > 0.0) || top_p > 1.0) return 1; /* exactly one rule */
    double m = -INFINITY;
    for (int v = 0; v < V; ++v) {
        if (isnan(l[v]) || l[v] == INFINITY) return 5;
        if (l[v] > m) m = l[v];
    }
    if (m == -INFINITY) return 5;
    double sum1 = 0.0;
    for (int v = 0; v < V; ++v) sum1 += exp(l[v] - m);
    double l1 = m + log(sum1); /* p is the model's own softmax over the WHOLE vocabulary */

    /* rank the tokens: larger logit first, lower id first among equals */
    ranked_t* rk = (ranked_t*)malloc(sizeof(ranked_t) * (size_t)V);
    for (int v = 0; v < V; ++v) { rk[v].l = l[v]; rk[v].v = v; }
    qsort(rk, (size_t)V, sizeof(ranked_t), by_logit_then_id);

    int k;
    double kmg = 1.0;
    if (top_k > 0) {
        k = top_k < V ? top_k : V;
    } else {
        /* nucleus on the proposal: the shortest run of ranked tokens whose mass under softmax(beta l) reaches top_p */
        double total = 0.0;
        for (int j = 0; j < V; ++j) total += exp(beta * (rk[j].l - m));
        double cum = 0.0;
        k = V;
        for (int j = 0; j < V; ++j) {
            double prev = cum;
            cum += exp(beta * (rk[j].l - m));
            if (cum >= top_p * total) {
                k = j + 1;
                kmg = fmin(fabs(cum / total - top_p), fabs(top_p - prev / total));
                break;
            }
        }
    }
    *k_own = k;
    if (force_k > 0) {
        /* how far an imposed size is from satisfying the rule (0 when it does): cum_{k-1} < top_p <= cum_k */
        if (top_k == 0 && force_k != k) {
            double total = 0.0, cum = 0.0, before = 0.0;
            for (int j = 0; j < V; ++j) total += exp(beta * (rk[j].l - m));
            for (int j = 0; j < force_k && j < V; ++j) { before = cum; cum += exp(beta * (rk[j].l - m)); }
            double short_by = top_p - cum / total;    /* > 0: the imposed set does not reach top_p */
            double over_by = before / total - top_p;  /* >= 0: one token fewer would have done */
            kmg = fmax(fmax(short_by, over_by), 0.0);
        }
        k = force_k < V ? force_k : V;
    }
    *k_used = k;
    *k_margin = kmg;

    unsigned char* in = (unsigned char*)calloc((size_t)V, 1);
    for (int j = 0; j < k; ++j) in[rk[j].v] = 1;
    free(rk);

    /* proposal q_S = softmax(beta l) restricted to S and renormalised; inverse CDF in vocabulary order over S */
    double total = 0.0;
    for (int v = 0; v < V; ++v) if (in[v]) total += exp(beta * (l[v] - m));
    double lb = beta * m + log(total);
    double target = U * total, cum = 0.0, below = 0.0, at = 0.0;
    int pick = -1, last_pos = -1;
    for (int v = 0; v < V; ++v) {
        if (!in[v]) continue;
        double e = exp(beta * (l[v] - m));
        double prev = cum;
        cum += e;
        if (e > 0.0) last_pos = v;
        if (pick < 0 && cum >= target) { pick = v; below = prev; at = cum; }
    }
    free(in);
    if (pick < 0) { pick = last_pos; below = at = total; }
    double mg = 1.0;
    if (below > 0.0) mg = fmin(mg, fabs(U - below / total));
    if (pick < last_pos) mg = fmin(mg, fabs(at / total - U));

    int tok = force_tok >= 0 ? force_tok : pick;
    double lp = l[tok] - l1;
    double lq = beta * l[tok] - lb;
    *y = tok;
    *y_own = pick;
    *logp_y = lp;
    *logq_y = lq;
    *log_omega = alpha_t * lp - lq; /* Eq. 7 with the proposal actually used */
    *margin = mg;
    return 0;
}

/* ------------------------------------------------------------------ */
/* Eq. 5                                                               */
/* ------------------------------------------------------------------ */
void orc_ess(const double* logW, int N, double* M, double* s1, double* s2, double* ess) {
    double mx = -INFINITY;
    for (int i = 0; i < N; ++i)
        if (logW[i] > mx) mx = logW[i];
    double a = 0.0, b = 0.0;
    for (int i = 0; i < N; ++i) {
        double w = exp(logW[i] - mx);
        a += w;
        b += w * w;
    }
    *M = mx;
    *s1 = a;
    *s2 = b;
    *ess = a * a / b; /* = 1 / sum_i (w_i / s1)^2 */
}

/* ------------------------------------------------------------------ */
/* systematic resampling                                               */
/* ------------------------------------------------------------------ */
void orc_systematic(const double* w, int N, double s1, double u0, int32_t* A, double* margin) {
    double* C = (double*)malloc(sizeof(double) * (size_t)N);
    double c = 0.0;
    for (int j = 0; j < N; ++j) {
        c += w[j];
        C[j] = c;
    }
    double mg = 1.0;
    for (int i = 0; i < N; ++i) {
        double pos = (u0 + (double)i) * s1; /* p_i * N * s1 */
        int a = N - 1;
        for (int j = 0; j < N; ++j) {
            if (C[j] * (double)N >= pos) {
                a = j;
                break;
            }
        }
        A[i] = a;
        double p = (u0 + (double)i) / (double)N;
        mg = fmin(mg, fabs(C[a] / s1 - p));
        if (a > 0) mg = fmin(mg, fabs(p - C[a - 1] / s1));
    }
    if (margin) *margin = mg;
    free(C);
}

/* ------------------------------------------------------------------ */
/* the other unbiased schemes of Appendix E ("Resampling Choices")     */
/* ------------------------------------------------------------------ */
/* first index j whose inclusive prefix C_j reaches `level` (both in the units of C), N-1 if rounding leaves none */
static int first_reaching(const double* C, int N, double level) {
    for (int j = 0; j < N; ++j)
        if (C[j] >= level) return j;
    return N - 1;
}
static void note_margin(const double* C, int N, double total, int a, double p, double* mg) {
    *mg = fmin(*mg, fabs(C[a] / total - p));
    if (a > 0) *mg = fmin(*mg, fabs(p - C[a - 1] / total));
}

/* stratified: one position per stratum, p_i = (i + u_i) / N with its own uniform u_i */
void orc_stratified(const double* w, int N, double s1, const double* u, int32_t* A, double* margin) {
    double* C = (double*)malloc(sizeof(double) * (size_t)N);
    double c = 0.0, mg = 1.0;
    for (int j = 0; j < N; ++j) { c += w[j]; C[j] = c; }
    for (int i = 0; i < N; ++i) {
        double pos = (u[i] + (double)i) * s1; /* p_i * N * s1, compared with C_j * N as in the systematic scheme */
        int a = N - 1;
        for (int j = 0; j < N; ++j)
            if (C[j] * (double)N >= pos) { a = j; break; }
        A[i] = a;
        note_margin(C, N, s1, a, (u[i] + (double)i) / (double)N, &mg);
    }
    if (margin) *margin = mg;
    free(C);
}

/* multinomial: N independent draws from Categorical(W), p_i = u_i */
void orc_multinomial(const double* w, int N, double s1, const double* u, int32_t* A, double* margin) {
    double* C = (double*)malloc(sizeof(double) * (size_t)N);
    double c = 0.0, mg = 1.0;
    for (int j = 0; j < N; ++j) { c += w[j]; C[j] = c; }
    for (int i = 0; i < N; ++i) {
        int a = first_reaching(C, N, u[i] * s1);
        A[i] = a;
        note_margin(C, N, s1, a, u[i], &mg);
    }
    if (margin) *margin = mg;
    free(C);
}

/* residual: floor(N W_j) copies of every j (in order of j), the remaining N - sum floors slots drawn
 * independently from the residual weights N W_j - floor(N W_j); u_m is the uniform of the m-th such draw */
void orc_residual(const double* w, int N, double s1, const double* u, int32_t* A, double* margin) {
    double* Cr = (double*)malloc(sizeof(double) * (size_t)N);
    double mg = 1.0, cr = 0.0;
    int D = 0;
    for (int j = 0; j < N; ++j) {
        double x = (double)N * w[j] / s1; /* expected offspring */
        double fl = floor(x);
        int n = (int)fl;
        mg = fmin(mg, fmin(x - fl, fl + 1.0 - x) / (double)N); /* how close the count is to flipping */
        for (int k = 0; k < n && D < N; ++k) A[D++] = j;
        cr += x - fl;
        Cr[j] = cr;
    }
    for (int m = 0; D < N; ++m, ++D) {
        int a = first_reaching(Cr, N, u[m] * cr);
        A[D] = a;
        if (cr > 0.0) note_margin(Cr, N, cr, a, u[m], &mg);
    }
    if (margin) *margin = mg;
    free(Cr);
}

void orc_resample(int kind, const double* w, int N, double s1, uint64_t seed, uint64_t g, uint64_t t, int32_t* A,
                  double* margin) {
    if (kind == ORC_RESAMPLE_SYSTEMATIC) {
        double u0 = orc_uniform(orc_hash5(seed, ORC_STREAM_RESAMPLE, g, t, 0));
        orc_systematic(w, N, s1, u0, A, margin);
        return;
    }
    double* u = (double*)malloc(sizeof(double) * (size_t)N);
    for (int i = 0; i < N; ++i) u[i] = orc_uniform(orc_hash5(seed, ORC_STREAM_RESAMPLE, g, t, (uint64_t)(1 + i)));
    if (kind == ORC_RESAMPLE_STRATIFIED) orc_stratified(w, N, s1, u, A, margin);
    else if (kind == ORC_RESAMPLE_MULTINOMIAL) orc_multinomial(w, N, s1, u, A, margin);
    else orc_residual(w, N, s1, u, A, margin);
    free(u);
}

void orc_slot_map(const int32_t* A, int N, int32_t* map) {
    int* off = (int*)calloc((size_t)N, sizeof(int));
    for (int i = 0; i < N; ++i) off[A[i]] += 1;
    for (int j = 0; j < N; ++j) map[j] = j; /* survivors keep their slot; dead ones overwritten below */
    int src = 0, used = 0; /* next source with surplus; copies of it already placed */
    for (int k = 0; k < N; ++k) {
        if (off[k] != 0) continue; /* slot k is dead: give it the next surplus offspring */
        while (src < N && off[src] - 1 <= used) {
            src += 1;
            used = 0;
        }
        map[k] = src;
        used += 1;
    }
    free(off);
}

/* ------------------------------------------------------------------ */
/* particle system                                                     */
/* ------------------------------------------------------------------ */
struct orc_ctx {
    int G, N, V, R, ramp, eos, T_max, t, resampler;
    double alpha, tau, kappa;
    uint64_t seed;
    int32_t* prompt_len;
    double *logW, *S, *log_inc, *logp_tok, *tok_margin, *ess, *logZ, *anc_margin;
    uint8_t* done;
    int32_t *len, *tok, *tok_own, *last_tok, *anc, *anc_own, *map, *resampled, *resampled_own;
    int32_t *tok_hist, *map_hist; /* [T_max][R] */
    int top_k;                    /* proposal restricted to the top of the row: at most one of the two is set */
    double top_p;
    const int32_t* force_k;       /* [R] sizes to impose at the next step (borrowed), or NULL */
    int32_t *k_used, *k_own;      /* [R] */
    double* k_margin;             /* [R] */
};

static void* zalloc(size_t n) { return calloc(n ? n : 1, 1); }

orc_ctx* orc_create(int G, int N, int V, double alpha, double tau, double kappa, int ramp,
                    uint64_t seed, int eos, int T_max, const int32_t* prompt_len) {
    if (G < 1 || N < 1 || V < 2 || alpha < 1.0 || tau <= 0.0 || kappa <= 0.0 || kappa > 1.0 ||
        ramp < 0 || eos < 0 || eos >= V || T_max < 1)
        return NULL;
    orc_ctx* c = (orc_ctx*)zalloc(sizeof(orc_ctx));
    c->G = G; c->N = N; c->V = V; c->R = G * N; c->ramp = ramp; c->eos = eos; c->T_max = T_max;
    c->alpha = alpha; c->tau = tau; c->kappa = kappa;
    size_t R = (size_t)c->R;
    c->prompt_len = (int32_t*)zalloc(sizeof(int32_t) * (size_t)G);
    if (prompt_len) memcpy(c->prompt_len, prompt_len, sizeof(int32_t) * (size_t)G);
    c->logW = (double*)zalloc(8 * R); c->S = (double*)zalloc(8 * R);
    c->log_inc = (double*)zalloc(8 * R); c->logp_tok = (double*)zalloc(8 * R);
    c->tok_margin = (double*)zalloc(8 * R);
    c->ess = (double*)zalloc(8 * (size_t)G); c->logZ = (double*)zalloc(8 * (size_t)G);
    c->anc_margin = (double*)zalloc(8 * (size_t)G);
    c->done = (uint8_t*)zalloc(R);
    c->len = (int32_t*)zalloc(4 * R); c->tok = (int32_t*)zalloc(4 * R);
    c->tok_own = (int32_t*)zalloc(4 * R); c->last_tok = (int32_t*)zalloc(4 * R);
    c->anc = (int32_t*)zalloc(4 * R); c->anc_own = (int32_t*)zalloc(4 * R);
    c->map = (int32_t*)zalloc(4 * R);
    c->resampled = (int32_t*)zalloc(4 * (size_t)G);
    c->resampled_own = (int32_t*)zalloc(4 * (size_t)G);
    c->tok_hist = (int32_t*)zalloc(4 * R * (size_t)T_max);
    c->map_hist = (int32_t*)zalloc(4 * R * (size_t)T_max);
    c->k_used = (int32_t*)zalloc(4 * R); c->k_own = (int32_t*)zalloc(4 * R); c->k_margin = (double*)zalloc(8 * R);
    orc_reset(c, seed);
    return c;
}

void orc_destroy(orc_ctx* c) {
    if (!c) return;
    free(c->prompt_len); free(c->logW); free(c->S); free(c->log_inc); free(c->logp_tok);
    free(c->tok_margin); free(c->ess); free(c->logZ); free(c->anc_margin); free(c->done);
    free(c->len); free(c->tok); free(c->tok_own); free(c->last_tok); free(c->anc);
    free(c->anc_own); free(c->map); free(c->resampled); free(c->resampled_own);
    free(c->tok_hist); free(c->map_hist); free(c->k_used); free(c->k_own); free(c->k_margin); free(c);
}

void orc_reset(orc_ctx* c, uint64_t seed) {
    c->seed = seed;
    c->t = 0;
    for (int g = 0; g < c->G; ++g) {
        c->logZ[g] = 0.0; c->ess[g] = (double)c->N; c->resampled[g] = 0; c->resampled_own[g] = 0;
        c->anc_margin[g] = 1.0;
        for (int i = 0; i < c->N; ++i) {
            int r = g * c->N + i;
            c->logW[r] = 0.0; /* W~_0 = 1 */
            c->S[r] = 0.0; c->done[r] = 0; c->len[r] = c->prompt_len[g];
            c->tok[r] = -1; c->tok_own[r] = -1; c->last_tok[r] = -1;
            c->anc[r] = i; c->anc_own[r] = i; c->map[r] = i;
            c->log_inc[r] = 0.0; c->logp_tok[r] = 0.0; c->tok_margin[r] = 1.0;
        }
    }
}

static double widen(const void* base, int dtype, int64_t idx) {
    if (dtype == ORC_F32) return (double)((const float*)base)[idx];
    if (dtype == ORC_F64) return ((const double*)base)[idx];
    uint32_t bits = (uint32_t)((const uint16_t*)base)[idx] << 16; /* bf16 = top half of an fp32 */
    float f;
    memcpy(&f, &bits, 4);
    return (double)f;
}

int orc_step(orc_ctx* c, const void* logits, int dtype, int64_t ld, const int32_t* force_tok,
             const int32_t* force_resample, const int32_t* force_anc) {
    if (c->t >= c->T_max) return 4;
    const int t = c->t + 1; /* token index of this step, 1-based */
    const int N = c->N, V = c->V, R = c->R;
    const double alpha_t = orc_alpha_at(c->alpha, c->ramp, t);
    const double alpha_prev = orc_alpha_at(c->alpha, c->ramp, t - 1);
    const double beta_t = orc_beta_at(c->alpha, c->tau, c->ramp, t);
    const double delta = alpha_t - alpha_prev; /* stage boundary before token t */
    int bad = 0;

    /* inner loop of Algorithm 1 over particles (independent, hence parallel) */
#pragma omp parallel for schedule(dynamic, 1) reduction(| : bad)
    for (int r = 0; r < R; ++r) {
        int g = r / N, i = r % N;
        /* boundary reweighting by (alpha_t - alpha_{t-1}) * log p(y_{1:t-1}); applies to every
           particle, finished ones included, so that the weights telescope to exponent alpha */
        c->logW[r] += delta * c->S[r];
        if (c->done[r]) { /* absorbing: emit EOS, factor 1, no cache growth */
            c->tok[r] = c->eos; c->tok_own[r] = c->eos;
            c->log_inc[r] = 0.0; c->logp_tok[r] = 0.0; c->tok_margin[r] = 1.0;
            continue;
        }
        double* l = (double*)malloc(sizeof(double) * (size_t)V);
        for (int v = 0; v < V; ++v) l[v] = widen(logits, dtype, (int64_t)r * ld + v);
        double U = orc_uniform(orc_hash5(c->seed, ORC_STREAM_TOKEN, (uint64_t)g, (uint64_t)t, (uint64_t)i));
        int y, y_own;
        double lp, lq, lw, l1, lb, mg;
        int rc;
        if (c->top_k > 0 || c->top_p > 0.0) {
            int ku, ko;
            double kmg;
            rc = orc_row_masked(l, V, beta_t, alpha_t, U, c->top_k, c->top_p, c->force_k ? c->force_k[r] : 0,
                                force_tok ? force_tok[r] : -1, &y, &y_own, &ku, &ko, &kmg, &lp, &lq, &lw, &mg);
            c->k_used[r] = ku; c->k_own[r] = ko; c->k_margin[r] = kmg;
        } else {
            rc = orc_row(l, V, beta_t, alpha_t, U, force_tok ? force_tok[r] : -1, &y, &y_own, &lp, &lq,
                         &lw, &l1, &lb, &mg);
        }
        free(l);
        if (rc) { bad |= 1; continue; }
        c->tok[r] = y; c->tok_own[r] = y_own; c->tok_margin[r] = mg;
        c->log_inc[r] = lw; c->logp_tok[r] = lp;
        c->logW[r] += lw;     /* W~_t = W~_{t-1} * p^alpha / q */
        c->S[r] += lp;        /* log p(y_{1:t}) */
        c->len[r] += 1;
        if (y == c->eos) c->done[r] = 1; /* after the weight update: EOS's own factor counts */
    }
    if (bad) return 5;

    int32_t* hist_tok = c->tok_hist + (size_t)(t - 1) * (size_t)R;
    int32_t* hist_map = c->map_hist + (size_t)(t - 1) * (size_t)R;
    memcpy(hist_tok, c->tok, sizeof(int32_t) * (size_t)R);

    double* w = (double*)malloc(sizeof(double) * (size_t)N);
    double* tmpd = (double*)malloc(sizeof(double) * (size_t)N);
    int32_t* tmpi = (int32_t*)malloc(sizeof(int32_t) * (size_t)N);
    uint8_t* tmpb = (uint8_t*)malloc((size_t)N);
    for (int g = 0; g < c->G; ++g) {
        double* lw = c->logW + (size_t)g * N;
        double M, s1, s2, ess;
        orc_ess(lw, N, &M, &s1, &s2, &ess);
        c->ess[g] = ess;
        int own = ess < c->kappa * (double)N; /* strict */
        c->resampled_own[g] = own;
        int fire = own;
        if (force_resample && force_resample[g] >= 0) fire = force_resample[g];
        c->resampled[g] = fire;
        int32_t* A = c->anc + (size_t)g * N;
        int32_t* A_own = c->anc_own + (size_t)g * N;
        int32_t* map = c->map + (size_t)g * N;
        c->anc_margin[g] = 1.0;
        if (!fire) {
            for (int i = 0; i < N; ++i) { A[i] = i; A_own[i] = i; map[i] = i; }
        } else {
            for (int i = 0; i < N; ++i) w[i] = exp(lw[i] - M);
            orc_resample(c->resampler, w, N, s1, c->seed, (uint64_t)g, (uint64_t)t, A_own, &c->anc_margin[g]);
            if (force_anc && force_anc[(size_t)g * N] >= 0)
                memcpy(A, force_anc + (size_t)g * N, sizeof(int32_t) * (size_t)N);
            else
                memcpy(A, A_own, sizeof(int32_t) * (size_t)N);
            orc_slot_map(A, N, map);
            c->logZ[g] += M + log(s1 / (double)N); /* log of the mean unnormalised weight */
            /* copy particle state by the map, then uniform weights */
            double* S = c->S + (size_t)g * N;
            uint8_t* dn = c->done + (size_t)g * N;
            int32_t* ln = c->len + (size_t)g * N;
            for (int k = 0; k < N; ++k) tmpd[k] = S[map[k]];
            memcpy(S, tmpd, sizeof(double) * (size_t)N);
            for (int k = 0; k < N; ++k) tmpb[k] = dn[map[k]];
            memcpy(dn, tmpb, (size_t)N);
            for (int k = 0; k < N; ++k) tmpi[k] = ln[map[k]];
            memcpy(ln, tmpi, sizeof(int32_t) * (size_t)N);
            for (int k = 0; k < N; ++k) lw[k] = 0.0;
        }
        for (int k = 0; k < N; ++k) {
            hist_map[(size_t)g * N + k] = map[k];
            c->last_tok[(size_t)g * N + k] = c->tok[(size_t)g * N + map[k]];
        }
    }
    free(w); free(tmpd); free(tmpi); free(tmpb);
    c->t = t;
    return 0;
}

void orc_reindex_tensor(void* dst, const void* src, int R, int H, int max_len, int D, int elem_size,
                        int64_t stride_row, int64_t stride_head, const int32_t* idx,
                        const int32_t* copy_len, const int32_t* copy_from) {
    const int in_place = (dst == src);
    for (int k = 0; k < R; ++k) {
        if (in_place && idx[k] == k) continue;
        int n = copy_len ? copy_len[k] : max_len;
        if (n > max_len) n = max_len;
        int f = copy_from ? copy_from[k] : 0; /* positions below f are left alone */
        if (f < 0) f = 0;
        if (n <= f) continue;
        for (int h = 0; h < H; ++h) {
            const char* s = (const char*)src + ((int64_t)idx[k] * stride_row + (int64_t)h * stride_head + (int64_t)f * D) * elem_size;
            char* d = (char*)dst + ((int64_t)k * stride_row + (int64_t)h * stride_head + (int64_t)f * D) * elem_size;
            memcpy(d, s, (size_t)(n - f) * (size_t)D * (size_t)elem_size);
        }
    }
}

void orc_select(orc_ctx* c, int32_t* out_tokens, int32_t* out_len, int32_t* out_index) {
    const int N = c->N, R = c->R, T = c->t;
    for (int g = 0; g < c->G; ++g) {
        const double* lw = c->logW + (size_t)g * N;
        double M, s1, s2, ess;
        orc_ess(lw, N, &M, &s1, &s2, &ess);
        double U = orc_uniform(orc_hash5(c->seed, ORC_STREAM_SELECT, (uint64_t)g, 0, 0));
        double target = U * s1, cum = 0.0;
        int I = N - 1;
        for (int i = 0; i < N; ++i) {
            cum += exp(lw[i] - M);
            if (cum >= target) { I = i; break; }
        }
        if (out_index) out_index[g] = I;
        int cur = I, first_eos = -1;
        int32_t* row = out_tokens ? out_tokens + (size_t)g * c->T_max : NULL;
        for (int t = T; t >= 1; --t) {
            cur = c->map_hist[(size_t)(t - 1) * R + (size_t)g * N + cur];
            int tok = c->tok_hist[(size_t)(t - 1) * R + (size_t)g * N + cur];
            if (row) row[t - 1] = tok;
            if (tok == c->eos) first_eos = t; /* going backwards: ends at the earliest */
        }
        if (row)
            for (int t = T; t < c->T_max; ++t) row[t] = -1;
        if (out_len) out_len[g] = first_eos > 0 ? first_eos : T;
    }
}

void orc_log_z_final(const orc_ctx* c, double* out) {
    for (int g = 0; g < c->G; ++g) {
        double M, s1, s2, ess;
        orc_ess(c->logW + (size_t)g * c->N, c->N, &M, &s1, &s2, &ess);
        out[g] = c->logZ[g] + M + log(s1 / (double)c->N);
    }
}

void orc_set_state(orc_ctx* c, const double* logW, const double* S, const uint8_t* done,
                   const int32_t* len) {
    size_t R = (size_t)c->R;
    if (logW) memcpy(c->logW, logW, 8 * R);
    if (S) memcpy(c->S, S, 8 * R);
    if (done) memcpy(c->done, done, R);
    if (len) memcpy(c->len, len, 4 * R);
}

int orc_t(const orc_ctx* c) { return c->t; }
const int32_t* orc_tokens(const orc_ctx* c) { return c->tok; }
const int32_t* orc_last_tokens(const orc_ctx* c) { return c->last_tok; }
const int32_t* orc_tokens_own(const orc_ctx* c) { return c->tok_own; }
const double* orc_tok_margin(const orc_ctx* c) { return c->tok_margin; }
const double* orc_log_weights(const orc_ctx* c) { return c->logW; }
const double* orc_log_inc(const orc_ctx* c) { return c->log_inc; }
const double* orc_logp_tok(const orc_ctx* c) { return c->logp_tok; }
const double* orc_cum_logp(const orc_ctx* c) { return c->S; }
const int32_t* orc_ancestors(const orc_ctx* c) { return c->anc; }
int orc_set_proposal_mask(orc_ctx* c, int top_k, double top_p) {
    if (!c || top_k < 0 || top_p < 0.0 || top_p > 1.0 || (top_k > 0 && top_p > 0.0)) return 1;
    c->top_k = top_k;
    c->top_p = top_p;
    return 0;
}
void orc_set_force_k(orc_ctx* c, const int32_t* force_k) { c->force_k = force_k; }
const int32_t* orc_k_used(const orc_ctx* c) { return c->k_used; }
const int32_t* orc_k_own(const orc_ctx* c) { return c->k_own; }
const double* orc_k_margin(const orc_ctx* c) { return c->k_margin; }
int orc_set_resampler(orc_ctx* c, int kind) {
    if (kind < 0 || kind > 3) return 1;
    c->resampler = kind;
    return 0;
}
const int32_t* orc_anc_own(const orc_ctx* c) { return c->anc_own; }
const double* orc_anc_margin(const orc_ctx* c) { return c->anc_margin; }
const int32_t* orc_slot_map_view(const orc_ctx* c) { return c->map; }
const int32_t* orc_resampled(const orc_ctx* c) { return c->resampled; }
const int32_t* orc_resampled_own(const orc_ctx* c) { return c->resampled_own; }
const double* orc_ess_view(const orc_ctx* c) { return c->ess; }
const double* orc_log_z(const orc_ctx* c) { return c->logZ; }
const int32_t* orc_lens(const orc_ctx* c) { return c->len; }
const uint8_t* orc_done(const orc_ctx* c) { return c->done; }
