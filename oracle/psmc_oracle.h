/*
 * Power-SMC CPU oracle -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, double-precision restatement of the per-token Power-SMC step
 * (Algorithm 1; Eq. 5 ESS; Eq. 7 incremental weight; Section 4.3 / Appendix B
 * exponent bridging; Appendix D absorbing EOS; the systematic-resampling rule
 * of the "Implementation details" paragraph of Section 6; Appendix C cache
 * reorder).  Sums run sequentially in index order; nothing is blocked, fused
 * or reordered.  It shares no code with the CUDA path and is imported only by
 * the tests, the smoke check and the CPU-baseline leg of the benchmark.
 *
 * Parity pins: every function here is pinned by the CPU test-suite against
 * closed forms, invariants, brute-force enumeration or a library routine --
 * except the absolute values of full-size trajectories, for which the paper
 * prints no worked example: "parity unpinned" for those; oracle <-> CUDA
 * agreement is the only check there.
 */
#ifndef PSMC_ORACLE_H
#define PSMC_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ORC_F32 = 0, ORC_BF16 = 1, ORC_F64 = 2 };
enum {
    ORC_STREAM_TOKEN = 1,    /* uniform for the token draw of (group, step, slot)   */
    ORC_STREAM_RESAMPLE = 2, /* offset u0 of systematic resampling of (group, step) */
    ORC_STREAM_SELECT = 3    /* uniform for the final Categorical(W) of a group     */
};

/* ---- counter-based randomness (a reading: the paper only says "sample") ---- */
uint64_t orc_sm64(uint64_t x);
uint64_t orc_hash5(uint64_t a, uint64_t b, uint64_t c, uint64_t d, uint64_t e);
double orc_uniform(uint64_t h); /* ((h >> 12) + 0.5) * 2^-52: exact, strictly in (0,1) */

/* ---- exponent schedule (Section 4.3, Appendix B) ---- */
double orc_alpha_at(double alpha, int ramp, int t);            /* alpha_t, t >= 0 */
double orc_beta_at(double alpha, double tau, int ramp, int t); /* alpha_t / (alpha * tau) */

/* ---- one row: log-softmax, tempered proposal, inverse-CDF draw, Eq. 7 ----
 * l[0..V) are the logits already widened to double.  Returns 0, or 5 when the
 * row has a NaN, a +inf, or no finite entry.  `force` >= 0 replaces the drawn
 * token (the draw is still made and reported in *y_own).  *margin is the
 * smaller distance, in CDF units, from U to the two CDF values that fence the
 * oracle's own token. */
int orc_row(const double* l, int V, double beta, double alpha_t, double U, int force,
            int* y, int* y_own, double* logp_y, double* logq_y, double* log_omega,
            double* L1, double* Lbeta, double* margin);

/* ---- one row with the proposal restricted to a set S of tokens (a reading: the paper names top-k and nucleus
 * only as decoding heuristics; used as an SMC proposal, the importance weight of Eq. 7 takes the proposal actually
 * sampled from, q_S(v) = exp(beta l_v) 1[v in S] / sum_{u in S} exp(beta l_u), while p stays the model's softmax
 * over the whole vocabulary; the target is thereby restricted to sequences the proposal can reach).
 * Tokens are ranked by logit, larger first, lower id first among equal logits; S = the first k of that ranking.
 *   top_k > 0, top_p == 0: k = min(top_k, V).
 *   top_k == 0, 0 < top_p <= 1: k = the smallest k whose ranked tokens hold at least top_p of the mass of
 *     softmax(beta l) (the proposal's own distribution, the one the temperature acts on).
 * Exactly one of the two must be set (returns 1 otherwise).  force_k > 0 imposes the size; *k_margin then tells by
 * how much (in mass units) that size misses the rule (0 if it satisfies it), and otherwise how close the oracle's
 * own decision was.  The draw is the inverse CDF over S in vocabulary order; *margin as in orc_row. */
int orc_row_masked(const double* l, int V, double beta, double alpha_t, double U, int top_k, double top_p,
                   int force_k, int force_tok, int* y, int* y_own, int* k_used, int* k_own, double* k_margin,
                   double* logp_y, double* logq_y, double* log_omega, double* margin);

/* ---- Eq. 5 on unnormalised log-weights ---- */
void orc_ess(const double* logW, int N, double* M, double* s1, double* s2, double* ess);

/* ---- systematic resampling: positions (u0+i)/N against the inclusive prefix
 * of the weights, first index reaching the position, clamped to N-1.
 * w are the unnormalised exp(logW - M); s1 their sum.  *margin = smallest
 * |position - prefix| met at a deciding comparison (in normalised units). */
void orc_systematic(const double* w, int N, double s1, double u0, int32_t* A, double* margin);

/* ---- the other unbiased schemes named in Appendix E.  u[i]: independent uniforms in (0,1).
 * stratified: position (i + u_i)/N in stratum i; multinomial: position u_i; residual: floor(N W_j) copies of
 * every j, in order of j, then the remaining slots drawn independently from the residual weights
 * N W_j - floor(N W_j) (u[m] for the m-th such slot).  Ancestors of multinomial and residual are not sorted.
 * *margin: smallest distance met at a deciding comparison (normalised units; for residual also the distance of
 * N W_j to the nearest whole number, over N). */
enum { ORC_RESAMPLE_SYSTEMATIC = 0, ORC_RESAMPLE_STRATIFIED = 1, ORC_RESAMPLE_MULTINOMIAL = 2, ORC_RESAMPLE_RESIDUAL = 3 };
void orc_stratified(const double* w, int N, double s1, const double* u, int32_t* A, double* margin);
void orc_multinomial(const double* w, int N, double s1, const double* u, int32_t* A, double* margin);
void orc_residual(const double* w, int N, double s1, const double* u, int32_t* A, double* margin);
/* ancestors of group g at step t under scheme `kind`: systematic takes u0 = H(seed, 2, g, t, 0), the others
 * u_i = H(seed, 2, g, t, 1 + i) */
void orc_resample(int kind, const double* w, int N, double s1, uint64_t seed, uint64_t g, uint64_t t, int32_t* A,
                  double* margin);

/* ---- hazard-free slot map from ancestors: survivors stay, dead slots (in
 * increasing order) take the surplus offspring (sources in increasing order) */
void orc_slot_map(const int32_t* A, int N, int32_t* map);

/* ---- particle system ---- */
typedef struct orc_ctx orc_ctx;

orc_ctx* orc_create(int G, int N, int V, double alpha, double tau, double kappa, int ramp,
                    uint64_t seed, int eos, int T_max, const int32_t* prompt_len /* [G] or NULL */);
void orc_destroy(orc_ctx*);
void orc_reset(orc_ctx*, uint64_t seed);
int orc_set_resampler(orc_ctx*, int kind); /* ORC_RESAMPLE_*; default systematic (Algorithm 1); 0 = ok */
/* restrict the proposal of every later step as in orc_row_masked (0, 0 = whole vocabulary, the paper's proposal) */
int orc_set_proposal_mask(orc_ctx*, int top_k, double top_p);
/* sizes to impose at the next steps, [G*N] (0 = the oracle's own), borrowed until replaced; NULL = none */
void orc_set_force_k(orc_ctx*, const int32_t* force_k);
const int32_t* orc_k_used(const orc_ctx*);  /* [R] size of S as applied at the last step */
const int32_t* orc_k_own(const orc_ctx*);   /* [R] the oracle's own size                 */
const double* orc_k_margin(const orc_ctx*); /* [R]                                       */

/* One token for every group.  logits: [G*N, V] row-major with row stride ld
 * elements, dtype ORC_*.  Hooks (each may be NULL): force_tok[G*N] (>=0 to
 * impose), force_resample[G] (0/1 to impose, -1 to let the oracle decide),
 * force_anc[G*N] (used for groups that resample; -1 in slot 0 of a group = own).
 * Returns 0 or 5 (numeric). */
int orc_step(orc_ctx*, const void* logits, int dtype, int64_t ld, const int32_t* force_tok,
             const int32_t* force_resample, const int32_t* force_anc);

/* Appendix C, flat form: one tensor [R, H, max_len, D] of elem_size bytes per
 * element, strides in elements; row k receives row idx[k] over positions
 * [0, copy_len[k]) (copy_len[k] = live length of the SOURCE row, which after
 * orc_step is the length recorded for slot k; NULL = max_len everywhere); the
 * rest of row k is left alone.  copy_from[k] (NULL = 0): positions below it are left alone too -- the form for
 * caches whose first positions (a prompt shared by the whole group) are the same in every row.  In place when dst == src: rows with idx[k]==k
 * are skipped and idx must be hazard-free (no row both read and written). */
void orc_reindex_tensor(void* dst, const void* src, int R, int H, int max_len, int D,
                        int elem_size, int64_t stride_row, int64_t stride_head,
                        const int32_t* idx, const int32_t* copy_len, const int32_t* copy_from);

/* Final draw I ~ Categorical(W_T) per group and back-trace of its tokens. */
void orc_select(orc_ctx*, int32_t* out_tokens /* [G, T_max] */, int32_t* out_len /* [G] */,
                int32_t* out_index /* [G] */);

/* ---- views of the state (owned by the ctx) ---- */
int orc_t(const orc_ctx*);
const int32_t* orc_tokens(const orc_ctx*);     /* [R] tokens of the last step, by the slot that drew them */
const int32_t* orc_last_tokens(const orc_ctx*); /* [R] last token of the particle now in each slot        */
const int32_t* orc_tokens_own(const orc_ctx*); /* [R] the oracle's own draw (before hook) */
const double* orc_tok_margin(const orc_ctx*);  /* [R]                                     */
const double* orc_log_weights(const orc_ctx*); /* [R] unnormalised log W after the step   */
const double* orc_log_inc(const orc_ctx*);     /* [R] log omega of the last step          */
const double* orc_logp_tok(const orc_ctx*);    /* [R] log p(y_t) of the last step         */
const double* orc_cum_logp(const orc_ctx*);    /* [R] S = sum_s log p(y_s)                */
const int32_t* orc_ancestors(const orc_ctx*);  /* [R] canonical A (identity if none)      */
const int32_t* orc_anc_own(const orc_ctx*);    /* [R] the oracle's own A (before hook)    */
const double* orc_anc_margin(const orc_ctx*);  /* [G]                                     */
const int32_t* orc_slot_map_view(const orc_ctx*); /* [R]                                  */
const int32_t* orc_resampled(const orc_ctx*);  /* [G] 0/1 as applied                      */
const int32_t* orc_resampled_own(const orc_ctx*); /* [G] the oracle's own decision        */
const double* orc_ess_view(const orc_ctx*);    /* [G] ESS before any resampling           */
const double* orc_log_z(const orc_ctx*);       /* [G] running log Z-hat                   */
const int32_t* orc_lens(const orc_ctx*);       /* [R] live KV length                      */
const uint8_t* orc_done(const orc_ctx*);       /* [R]                                     */
/* log Z-hat including the not-yet-reset weights: logZ + M + log(s1/N) */
void orc_log_z_final(const orc_ctx*, double* out /* [G] */);
/* overwrite state (for unit-level parity on identical inputs) */
void orc_set_state(orc_ctx*, const double* logW, const double* S, const uint8_t* done,
                   const int32_t* len);

#ifdef __cplusplus
}
#endif
#endif
