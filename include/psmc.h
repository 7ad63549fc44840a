/*
 * psmc -- the per-token Power-SMC step on one NVIDIA B200 (sm_100a), C-ABI.
 *
 * Everything here runs in hand-written CUDA kernels; there is no CPU fallback.
 * The calls follow Algorithm 1 of the paper: N particles per prompt ("group"),
 * G independent groups, R = G*N rows.  One decoded token is one psmc_step()
 * (the loop body of Algorithm 1: proposal, draw, weight update of Eq. 7, EOS
 * handling, normalisation and ESS of Eq. 5, ESS-triggered systematic
 * resampling) followed by psmc_reindex_kv() (its cache reorder, Appendix C) and, after the
 * last token, psmc_select() (its output step).
 *
 * Conventions
 *   - Every call returns a psmc_status; nothing throws or aborts.
 *   - "DEVICE" pointers are CUDA global-memory addresses on the context's
 *     device; "HOST" pointers are ordinary process memory.  The caller owns
 *     every buffer it passes; the context owns its own state.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     All work is stream-ordered and asynchronous unless a call says it syncs.
 *     Calls on one context must be issued on one stream (or be ordered by the
 *     caller): they share the context's scratch memory.
 *   - Errors the host can see (null pointer, size out of range, step beyond
 *     T_max) return at once and enqueue nothing.  Errors only the device can
 *     see (a NaN or +inf logit, a row without finite logits, a hazardous gather
 *     vector, a bounded wait that ran out) set a sticky device status word that
 *     psmc_sync_status() returns; the kernels never trap.
 *   - No kernel waits for another CTA or another kernel: the only device-side
 *     waits are for bulk copies into a CTA's own shared memory (bounded; on
 *     expiry PSMC_E_TIMEOUT is raised, the affected rows get token -1 and the
 *     kernel ends normally) and for warps of the same CTA.  Contexts may
 *     therefore share a GPU, on any streams, with each other and with other
 *     kernels.  After any device-detected error the context's counters are
 *     consistent again at the end of the launch; psmc_reset() clears the
 *     status word and restarts the run.
 *   - Randomness is a counter hash, so a run is a pure function of (seed,
 *     inputs): sm64(x) is the splitmix64 finaliser of x + 0x9E3779B97F4A7C15;
 *     H(a,b,c,d,e) = sm64(sm64(sm64(sm64(sm64(a)^b)^c)^d)^e); a uniform is
 *     ((H >> 12) + 0.5) * 2^-52.  Streams: H(seed,1,group,t,slot) token draw,
 *     H(seed,2,group,t,0) resampling offset, H(seed,3,group,0,0) final draw.
 */
#ifndef PSMC_H
#define PSMC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct psmc_ctx psmc_ctx; /* opaque, owned by the library */

typedef enum {
    PSMC_OK = 0,
    PSMC_E_INVAL = 1,   /* bad argument                                            */
    PSMC_E_NOMEM = 2,   /* device or host allocation failed                        */
    PSMC_E_CUDA = 3,    /* a CUDA runtime call failed                              */
    PSMC_E_STATE = 4,   /* call out of order (e.g. step beyond T_max)              */
    PSMC_E_NUMERIC = 5, /* NaN / +inf logit, or a row with no finite logit         */
    PSMC_E_TIMEOUT = 6, /* a bounded device-side wait (for a bulk copy) gave up    */
    PSMC_E_HAZARD = 7,  /* in-place gather vector reads a row that is also written */
    PSMC_E_TOO_LARGE = 8 /* problem needs more than the fixed scratch of psmc_logits_pass_static */
} psmc_status;

typedef enum { PSMC_F32 = 0, PSMC_BF16 = 1 } psmc_dtype;

/* Resampling schemes (Appendix E, "Resampling Choices": any unbiased scheme preserves the target). */
typedef enum {
    PSMC_RESAMPLE_SYSTEMATIC = 0,  /* Algorithm 1, Section 6: positions (u0 + i)/N, one uniform per group and step */
    PSMC_RESAMPLE_STRATIFIED = 1,  /* positions (u_i + i)/N, one uniform per particle                            */
    PSMC_RESAMPLE_MULTINOMIAL = 2, /* positions u_i: N independent draws from Categorical(W)                     */
    PSMC_RESAMPLE_RESIDUAL = 3     /* floor(N W_j) copies of j, the rest drawn from the residual weights          */
} psmc_resampler;

/* ------------------------------------------------------------------------- */
/* Context (inputs of Algorithm 1: alpha, N, kappa, T_max, proposal)          */
/* ------------------------------------------------------------------------- */

/* One group.  N particles (1..1024), V vocabulary size (>= 2), alpha >= 1 the
 * power exponent of Eq. 1, tau > 0 the proposal temperature at full alpha
 * (Corollary 1: tau = 1/alpha is the variance-optimal choice), ess_thresh =
 * kappa in (0,1] (resample when ESS < kappa*N, Algorithm 1), ramp = T_ramp tokens of
 * linear exponent bridging (Section 4.3; 0 = off), eos_id in [0,V).  History
 * capacity T_max = 4096, initial KV length 0.  Allocates device state on the
 * current CUDA device. */
psmc_status psmc_init(psmc_ctx** out, int N, int V, float alpha, float tau, float ess_thresh,
                      int ramp, uint64_t seed, int eos_id);

/* G independent groups with per-group initial KV length (HOST array [G], may
 * be NULL = 0) and history capacity T_max steps. */
psmc_status psmc_init_batched(psmc_ctx** out, int G, int N, int V, float alpha, float tau,
                              float ess_thresh, int ramp, uint64_t seed, int eos_id, int T_max,
                              const int32_t* prompt_len_host);

/* Scheme used by the following steps (default PSMC_RESAMPLE_SYSTEMATIC).  Uniforms: H(seed,2,group,t,0) for the
 * systematic offset, H(seed,2,group,t,1+i) for particle (or residual draw) i of the others.  For multinomial and
 * residual resampling the ancestor vector is in drawing order, not sorted. */
psmc_status psmc_set_resampler(psmc_ctx*, psmc_resampler kind);

/* Restrict the proposal of the following steps to a set S of tokens per row.  (The paper's proposal is the whole
 * tempered distribution of Corollary 1; it names top-k and nucleus sampling only as decoding heuristics.  Used as an
 * SMC proposal they enter Eq. 7 as the distribution actually sampled from:
 *   q_S(v) = exp(beta_t l_v) / sum_{u in S} exp(beta_t l_u) for v in S,  log omega = alpha_t log p(y) - log q_S(y),
 * with p the model's softmax over the WHOLE vocabulary; the particle system then targets p^alpha restricted to the
 * sequences the proposal can reach.)  Tokens rank by logit, larger first, lower id first among equal logits (-0 and
 * +0 are equal); S is the first k of that ranking:
 *   top_k > 0, top_p == 0:      k = min(top_k, V)
 *   top_k == 0, 0 < top_p <= 1: k = the smallest k whose ranked tokens hold a share top_p of softmax(beta_t l)
 *                               (masses are compared as 2^-40 fixed-point fractions of the largest token's mass)
 *   0, 0:                       the whole vocabulary again (the default)
 * PSMC_E_INVAL for anything else.  The draw is the inverse CDF over S in vocabulary order with the same uniforms as
 * the unrestricted step.  psmc_mask_sizes() holds k of every row that was live at the last step.  The restricted
 * step runs as a pass of its own (one CTA per row: a radix search over the logits' bit patterns for the k-th ranked
 * key, then the masked sums), not combinable with the sharded step (PSMC_E_STATE there). */
psmc_status psmc_set_proposal_mask(psmc_ctx*, int top_k, double top_p);

psmc_status psmc_destroy(psmc_ctx*);                 /* syncs the device, frees everything   */
psmc_status psmc_reset(psmc_ctx*, uint64_t seed);    /* t=0, weights 1, S=0, done=0; syncs    */

/* ------------------------------------------------------------------------- */
/* One token (the loop body of Algorithm 1 without the cache move)            */
/* ------------------------------------------------------------------------- */

/* logits: DEVICE [R, V] row-major, row stride `ld` elements (>= V), dtype dt.
 * Rows whose start is 16-byte aligned take the 128-bit load path (base pointer
 * 16-byte aligned and ld*sizeof(elem) a multiple of 16); otherwise a scalar
 * path is used.  Finished rows are not read.  On return (stream-ordered) the
 * views below hold this step's results. */
psmc_status psmc_step(psmc_ctx*, const void* logits, psmc_dtype dt, int64_t ld, void* stream);

/* The same step fed from HOST memory: copies [R,V] logits (row stride ld) to a
 * staging buffer owned by the context, runs the step, copies the R drawn
 * tokens (as seen by each slot after resampling, i.e. the next LM input) back
 * to tokens_out_host, and synchronises the stream.  The logits travel on a stream of the context's own, so the copy
 * overlaps work still queued on `stream` (the previous token's cache move).  Pinned host memory makes
 * the copies asynchronous with respect to the host until that final sync. */
psmc_status psmc_step_host(psmc_ctx*, const void* logits_host, psmc_dtype dt, int64_t ld,
                           int32_t* tokens_out_host, void* stream);

/* Stateless form of the logit pass alone (Eq. 7 with the proposal of
 * Corollary 1): for each row r with done[r]==0 computes L1 = logsumexp(l),
 * Lb = logsumexp(beta*l), draws y = min{v : sum_{u<=v} exp(beta*l_u) >= U_r *
 * sum_all} and writes tok[r] = y, logp[r] = l_y - L1, loginc[r] = alpha_t *
 * logp[r] - (beta*l_y - Lb).  All pointers DEVICE.  u: [R] uniforms in (0,1).
 * done may be NULL (all live); rows with done[r]!=0 are left untouched.
 * scratch: at least psmc_logits_pass_scratch_bytes(R, V) bytes, 256-byte
 * aligned, contents irrelevant on entry (it carries per-span partial sums from
 * the streaming kernel to the finishing kernel of this call); status_word: one
 * int32, sticky PSMC_E_* code (0 = fine).  A flagged row gets tok = -1. */
size_t psmc_logits_pass_scratch_bytes(int R, int V);
psmc_status psmc_logits_pass(const void* logits, psmc_dtype dt, int R, int V, int64_t ld,
                             double beta, double alpha_t, const double* u, const uint8_t* done,
                             void* scratch, size_t scratch_bytes, int32_t* tok, double* logp,
                             double* loginc, int32_t* status_word, void* stream);

/* The logit pass for callers that cannot allocate device memory.  (The paper
 * has no counterpart: this is a packaging variant of psmc_logits_pass.)
 *
 * Some hosts of this library are handed raw input and output pointers and
 * nothing else: a custom-op hook inside a serving runtime whose memory pool
 * belongs to the runtime, a plug-in running under a framework that forbids
 * cudaMalloc while its own allocator is active (cudaMalloc synchronises the
 * device and would stall every other stream), a real-time loop with a "no
 * allocation after start-up" rule.  They have nowhere to get the scratch
 * buffer psmc_logits_pass asks for, and psmc_init is closed to them too.
 *
 * This entry point takes the same inputs and outputs as psmc_logits_pass but
 * no scratch: the per-span partial sums go to a fixed array of
 * PSMC_STATIC_SCRATCH_BYTES that is part of the library's device image, so
 * every GPU that loads the library carries it (4 MiB) until the process exits.
 * The call itself performs no cudaMalloc, cudaFree or other allocating call.
 *
 *   - Limit: psmc_logits_pass_scratch_bytes(R, V) must not exceed
 *     PSMC_STATIC_SCRATCH_BYTES (16 bytes per span of 1024-4096 logits per row;
 *     e.g. 512 rows x 128256 logits need 262,144 bytes).  Larger problems are
 *     refused with PSMC_E_TOO_LARGE and nothing is enqueued.
 *   - First call on each device: looks up the array's device address (a
 *     runtime symbol query, with that device current) and caches it.  Make that
 *     first call outside any stream capture.
 *   - One array per device, shared by every call and every stream: two calls
 *     that overlap on the GPU (different streams, or different host threads
 *     without ordering) race on it and corrupt each other's results.  Issue
 *     calls on one stream or order them yourself.  The array keeps the previous
 *     call's contents; nothing in it needs clearing, because each call
 *     overwrites every entry it later reads.
 * Results are identical to psmc_logits_pass on the same inputs. */
#define PSMC_STATIC_SCRATCH_BYTES (4u << 20)
psmc_status psmc_logits_pass_static(const void* logits, psmc_dtype dt, int R, int V, int64_t ld,
                                    double beta, double alpha_t, const double* u,
                                    const uint8_t* done, int32_t* tok, double* logp, double* loginc,
                                    int32_t* status_word, void* stream);

/* ------------------------------------------------------------------------- */
/* KV-cache reindex (Algorithm 1's cache reorder, Appendix C)                  */
/* ------------------------------------------------------------------------- */
typedef struct {
    int n_layers;
    void* const* k;        /* HOST array [n_layers] of DEVICE pointers, each [R, H, max_len, D] */
    void* const* v;        /* same for values                                                   */
    int n_kv_heads;        /* H */
    int head_dim;          /* D */
    int max_len;
    psmc_dtype dt;
    int64_t stride_row;    /* elements between rows (particles)                    */
    int64_t stride_head;   /* elements between heads; (position, dim) is contiguous */
    int skip_shared_prompt; /* src only, step maps only: nonzero = leave positions below the group's prompt length alone */
} psmc_kv_desc;

/* Applies the slot map of the most recent step to caller-owned caches: for
 * every layer, K and V, head h and slot k with map[k] != k, positions
 * [0, len) of row map[k] are copied onto row k, where len is the live length
 * of the source row; the tail of row k is not touched.  Groups that did not
 * resample move nothing, and a step without any resampling returns after
 * reading one device counter (no host sync either way).
 *   dst == NULL: in place on src.  The step's own slot map never reads a row it
 *     writes.  idx_override (DEVICE [R], may be NULL) replaces the map by an
 *     arbitrary gather vector with ROW indices in [0,R) and full-length copies
 *     (max_len positions); in place it must be hazard-free, else
 *     PSMC_E_HAZARD is raised in the status word and nothing is written.
 *   dst != NULL: out-of-place gather dst[k] = src[idx[k]] for every k (also
 *     idx[k]==k), i.e. index_select on the particle dimension.
 * src->skip_shared_prompt: all particles of a group start from the same prompt, so the first prompt_len positions
 *   of their rows hold the same keys and values; when the caller vouches for that (the rows were prefilled with one
 *   prompt per group) the copy of a row starts at the group's prompt length given to psmc_init_batched and only
 *   generated positions move.  Ignored with idx_override.
 * The bulk-copy (TMA) path needs 16-byte aligned row/head starts and
 * head_dim*sizeof(elem) a multiple of 16; otherwise a plain-load path runs. */
psmc_status psmc_reindex_kv(psmc_ctx*, const psmc_kv_desc* src, const psmc_kv_desc* dst,
                            const int32_t* idx_override, void* stream);

/* ------------------------------------------------------------------------- */
/* Paged KV cache with copy-on-write resampling (Appendix C on a block table)  */
/* ------------------------------------------------------------------------- */
/* The cache reorder of Algorithm 1 asks that slot k hold the cache of its ancestor.  With the cache cut into
 * blocks of block_len positions that are reached through a per-row block table, a duplicated particle can SHARE
 * its ancestor's full blocks (a table entry and a reference count instead of a copy); only the last, partly
 * filled block is copied, because both particles go on appending to it.  The bytes moved per rewritten slot drop
 * from len to less than block_len positions.  The result is the same cache, read through the table:
 * position p of row r lives in block table[r][p / block_len] at offset p % block_len.
 *
 * The context owns the table [R, max_blocks_per_row] (-1 = no block), the reference counts [n_blocks] and the
 * free list; the caller owns the pools.  psmc_kv_paged_create sizes them and gives every row the blocks of its
 * prompt (lengths of psmc_init_batched): with share_prompt != 0 the full blocks of a prompt are shared by the N
 * rows of its group and only a partly filled last block is private; the caller then writes the prompt's keys and
 * values through the table (once per group for shared blocks).  Invariant kept by every call: a partly filled
 * block has exactly one owner.  Running out of blocks raises PSMC_E_NOMEM in the status word.  Synchronises. */
psmc_status psmc_kv_paged_create(psmc_ctx*, int n_blocks, int block_len, int max_blocks_per_row, int share_prompt);

/* Before the language model writes position len[r] of every live row: rows whose next position starts a new block
 * get one from the free list, unless they hold it already.  Stream-ordered.  Needed once, after
 * psmc_kv_paged_create and the prefill: psmc_reindex_kv_paged does the same for the token that follows it (see
 * there), and a call that finds every row provided for changes nothing. */
psmc_status psmc_kv_paged_append(psmc_ctx*, void* stream);

/* At most 64 layers per call; pools 16-byte aligned with head_dim*sizeof(elem) a multiple of 16. */
typedef struct {
    int n_layers;
    void* const* k;      /* HOST array [n_layers] of DEVICE pointers, each pool [n_blocks, H, block_len, D] contiguous */
    void* const* v;
    int n_kv_heads;      /* H */
    int head_dim;        /* D */
    psmc_dtype dt;
} psmc_kv_pools;

/* Applies the slot map of the most recent step: every rewritten slot gives its blocks back, takes a reference to
 * each full block of its ancestor and a private copy of the ancestor's partly filled last block (all layers, K and
 * V, all heads).  Groups that did not resample change nothing.  Unless the step was the last one the context can
 * take (T_max), every live row is then given the block its next position needs, exactly as psmc_kv_paged_append
 * would (same errors), so that a token costs three launches here and none for the append.  Stream-ordered, no host
 * synchronisation. */
psmc_status psmc_reindex_kv_paged(psmc_ctx*, const psmc_kv_pools* pools, void* stream);

/* DEVICE views of the paging state (valid until psmc_destroy or the next psmc_kv_paged_create). */
const int32_t* psmc_kv_paged_table(psmc_ctx*);      /* [R, max_blocks_per_row] */
const int32_t* psmc_kv_paged_refcount(psmc_ctx*);   /* [n_blocks]              */
const int32_t* psmc_kv_paged_free_count(psmc_ctx*); /* [1] blocks on the free list */

/* ------------------------------------------------------------------------- */
/* Output (last step of Algorithm 1)                                          */
/* ------------------------------------------------------------------------- */

/* Per group draws I ~ Categorical(W) from the current weights and writes the
 * token string of particle I.  DEVICE outputs: out_tokens [G, T_max] (the
 * first t entries are tokens, EOS repeated after termination, the rest -1),
 * out_len [G] (tokens up to and including the first EOS, else t), out_index
 * [G] (the slot I).  Any of them may be NULL. */
psmc_status psmc_select(psmc_ctx*, int32_t* out_tokens, int32_t* out_len, int32_t* out_index,
                        void* stream);

/* ------------------------------------------------------------------------- */
/* Views of the context state: DEVICE pointers, valid until psmc_destroy;      */
/* contents are those of the most recent step once the stream has reached it.  */
/* ------------------------------------------------------------------------- */
const int32_t* psmc_tokens(psmc_ctx*);       /* [R] token drawn by each slot in the last step            */
const int32_t* psmc_last_tokens(psmc_ctx*);  /* [R] last token of the particle now in each slot          */
const double*  psmc_log_weights(psmc_ctx*);  /* [R] unnormalised log W after the step (0 after resample) */
const double*  psmc_log_inc(psmc_ctx*);      /* [R] log omega of the last step (Eq. 7)                   */
const double*  psmc_logp_tok(psmc_ctx*);     /* [R] log p(y_t) of the last step                          */
const double*  psmc_cum_logp(psmc_ctx*);     /* [R] S = log p(y_{1:t})                                   */
const int32_t* psmc_ancestors(psmc_ctx*);    /* [R] systematic-resampling ancestors A (identity if none) */
const int32_t* psmc_slot_map(psmc_ctx*);     /* [R] hazard-free map applied to state and KV              */
const int32_t* psmc_resampled(psmc_ctx*);    /* [G] 0/1                                                  */
const double*  psmc_ess(psmc_ctx*);          /* [G] ESS of Eq. 5 before resampling                       */
const double*  psmc_log_z(psmc_ctx*);        /* [G] running log of the normaliser estimate               */
const int32_t* psmc_mask_sizes(psmc_ctx*);    /* [R] size of the proposal's support at the last step (psmc_set_proposal_mask) */
const int32_t* psmc_lens(psmc_ctx*);         /* [R] live KV length                                       */
const uint8_t* psmc_done(psmc_ctx*);         /* [R] finished flags (ask again after each step: steps read one array
                                                    and write another, and the two alternate)                 */
const int32_t* psmc_move_count(psmc_ctx*);   /* [1] slots rewritten by the last step's maps (ask again after each step:
                                                    the counter alternates between two words)                */

int psmc_step_index(const psmc_ctx*);        /* t: tokens decoded so far                                 */
int psmc_rows(const psmc_ctx*);              /* R                                                        */

/* Overwrite particle state from HOST arrays [R] (any may be NULL = keep);
 * synchronises.  For unit tests and for resuming a saved run. */
psmc_status psmc_set_state(psmc_ctx*, const double* log_w, const double* cum_logp,
                           const uint8_t* done, const int32_t* lens);

/* ------------------------------------------------------------------------- */
/* The step with the vocabulary split over P ranks                            */
/* ------------------------------------------------------------------------- */

/* A tensor-parallel LM head leaves rank p with columns [v0_p, v0_p + V_p) of every logit row (the shards tile the
 * vocabulary in rank order).  The proposal of Corollary 1 and the weight of Eq. 7 need two row sums and one token's
 * logit, so the step splits into three calls around two small exchanges that the CALLER performs (an all-gather
 * over its process group; this library does no communication):
 *
 *   psmc_shard_sweep   reads the local columns once and writes one triple per row to triples_out (DEVICE [R][3]
 *                      doubles: the shard's reference exponent C_p, a whole number, then sum 2^{x - C_p} and
 *                      sum 2^{beta_t (x - C_p)} over its columns, x = logit * log2 e; zeros for finished rows)
 *   -- all-gather --   all_triples: DEVICE [P][R][3], the ranks' triples in rank order, identical on every rank
 *   psmc_shard_locate  every rank derives the same row totals, target mass U * Sb and owner (the first rank whose
 *                      inclusive mass prefix reaches the target); the owner finds the token among its columns.
 *                      picks_out: DEVICE [R]; tok = token id in the WHOLE vocabulary (v0 + local column) and
 *                      its logit on the owner, tok = -1 elsewhere and for finished rows
 *   -- all-gather --   all_picks: DEVICE [P][R] in rank order
 *   psmc_shard_finish  log p(y), log omega (Eq. 7) and the rest of the step (weights, ESS, trigger, resampling,
 *                      slot map) exactly as psmc_step does, identically on every rank
 *
 * Every rank creates its context with the same parameters (V = the whole vocabulary, the same seed) and the same
 * sequence of calls, so the replicated particle state stays bit-identical across ranks and psmc_reindex_kv /
 * psmc_select work unchanged on each rank's share of the cache.  The token drawn is the one psmc_step draws from
 * the whole row up to the rounding of the partial sums (the inverse CDF runs over the vocabulary in its natural
 * order).  The three calls must come in this order (PSMC_E_STATE otherwise); the logits of the sweep must stay
 * untouched until psmc_shard_locate has run.  V_local >= 2, sum over ranks = V; v0 >= 0, v0 + V_local <= V;
 * 1 <= P <= 1024.  A shard whose columns are all -inf is fine.  Alignment rules for the fast path as in psmc_step,
 * applied to the shard's first column. */
typedef struct {
    int32_t tok;   /* token id in the whole vocabulary, -1 = not this rank's row */
    float logit;   /* the token's logit (bf16 and fp32 are both exact in a float) */
} psmc_shard_pick;
psmc_status psmc_shard_sweep(psmc_ctx*, const void* logits_local, psmc_dtype dt, int64_t ld, int V_local,
                             double* triples_out, void* stream);
psmc_status psmc_shard_locate(psmc_ctx*, int v0, const double* all_triples, int P, int rank,
                              psmc_shard_pick* picks_out, void* stream);
psmc_status psmc_shard_finish(psmc_ctx*, const double* all_triples, const psmc_shard_pick* all_picks, int P,
                              void* stream);

/* ------------------------------------------------------------------------- */
/* The step fed one vocabulary tile at a time                                 */
/* ------------------------------------------------------------------------- */

/* For a caller whose LM-head GEMM produces the logits of one vocabulary tile [R, width] at a time and never writes
 * the [R, V] block to memory (the tile is consumed while it is still in L2).  The proposal of Corollary 1 and the
 * weight of Eq. 7 need two row sums, which can be accumulated tile by tile, and the logits around the drawn token,
 * which are only known to matter once the sums are complete; so the step is three kinds of calls:
 *
 *   psmc_tiles_feed    once per tile, in vocabulary order (v0 = 0, width, 2 width, ...; all tiles of one width but
 *                      possibly the last; v0 + width <= V): reads the tile once and keeps one triple per row
 *                      (reference exponent, sum 2^{x - c}, sum 2^{beta_t (x - c)}).  tile_logits: DEVICE [R, width],
 *                      row stride ld elements; it may be overwritten as soon as the call's work on `stream` is done.
 *   psmc_tiles_need    after the tile that ends at V: first_column_out (DEVICE int32 [R]) receives, per row, the first
 *                      column of the tile that holds the row's target mass U * sum (-1 for a finished row).
 *   psmc_tiles_finish  row_tiles: DEVICE [R, >= tile width], row stride ld: row r holds the logits of columns
 *                      first_column[r] ... of ITS row again (recomputed by the caller: one tile per row, 1 / n_tiles
 *                      of the GEMM), with -inf in columns beyond the vocabulary (last tile) and anything in finished
 *                      rows.  Draws the token inside the tile, forms log p(y) and log omega (Eq. 7) from the
 *                      accumulated sums and runs the rest of the step exactly as psmc_step does.
 *
 * The drawn token is the one psmc_step draws from the whole row up to the rounding of the partial sums (the inverse
 * CDF runs over the vocabulary in its natural order).  Calls out of order return PSMC_E_STATE; not combinable with
 * psmc_set_proposal_mask.  At most 1024 tiles. */
psmc_status psmc_tiles_feed(psmc_ctx*, const void* tile_logits, psmc_dtype dt, int64_t ld, int v0, int width,
                            void* stream);
psmc_status psmc_tiles_need(psmc_ctx*, int32_t* first_column_out, void* stream);
psmc_status psmc_tiles_finish(psmc_ctx*, const void* row_tiles, psmc_dtype dt, int64_t ld, void* stream);

/* Snapshot of a run, for checkpointing and for moving a run to another context.  Because all randomness is a
 * counter hash of (seed, group, step, slot), a context that loads a snapshot continues bit for bit as the one that
 * saved it would have.  The snapshot holds the particle state, the results of the last step and the ancestry log
 * up to the current step; caches (dense or paged, with their tables) are the caller's to save, and the move list
 * of a step does not travel: take the snapshot after the step's cache move.  psmc_state_save
 * writes psmc_state_bytes() bytes to HOST memory; psmc_state_load needs a context created with the same G, N, V,
 * T_max and per-group prompt lengths (PSMC_E_INVAL otherwise, nothing loaded) and takes over alpha, tau, kappa, ramp, eos, seed, resampler and
 * the step counter from the snapshot.  Both synchronise the device. */
size_t psmc_state_bytes(const psmc_ctx*);
psmc_status psmc_state_save(psmc_ctx*, void* host_buf, size_t bytes);
psmc_status psmc_state_load(psmc_ctx*, const void* host_buf, size_t bytes);

/* Profiling aid.  on = 1: every kernel launched by psmc_step / psmc_step_host / psmc_reindex_kv is bracketed by
 * CUDA events on the caller's stream.  on = 2: one bracket around the kernels of a psmc_step (they then keep
 * their chained launches) and one around every reindex kernel.  on = 0: off.  psmc_timing_read waits for the
 * recorded events, adds up the device time per bracket kind (HOST arrays of 3: [0] logit pass, or with on = 2 the
 * whole step; [1] weights/ESS/resampling when it is a kernel of its own; [2] KV reindex; milliseconds and
 * bracket counts) and clears the record.
 * Independently of this, every call that launches kernels (psmc_step, psmc_step_host, psmc_reindex_kv, the paged,
 * sharded and tile-fed calls, psmc_select, psmc_reset) opens an NVTX range named after itself on the calling
 * thread for the duration of the call, so that timelines of NVTX-aware tools show which call a kernel belongs to. */
psmc_status psmc_timing_enable(psmc_ctx*, int on);
psmc_status psmc_timing_read(psmc_ctx*, double* ms_out, int64_t* launches_out);

/* Diagnostic, host only (no GPU, no context): how the one-kernel form of psmc_step (Algorithm 1's loop body without the
 * cache move) deals a block of R rows x V logits to its CTAs.  Rows are cut into granules of 512 bytes; CTA b streams
 * the granules [shares_out[b], shares_out[b + 1]) of the block in row-major order.  layout_out: HOST array of 8:
 * [0] 1 if the shape fits the one-kernel form (16-byte aligned rows assumed), else 0; [1] CTAs; [2] streaming warps per
 * CTA; [3] granules per row; [4] bound on the rows one CTA's share meets; [5] CTAs per row when every row is dealt to
 * CTAs of its own, else 0; [6] bytes of a row that bulk copies fetch; [7] logits of a row after them.  shares_out: HOST
 * array of at least CTAs + 1 entries (shares_cap says how many there are), or NULL.  PSMC_E_INVAL: bad arguments or an
 * array too short.  psmc_step_share_of: the CTA whose share holds a granule, -1 for a granule outside the block or a
 * shape that does not fit.  (The paper has no counterpart: this is the kernel's own work division, exposed for tests.) */
psmc_status psmc_step_layout(int R, int V, psmc_dtype dt, int32_t* layout_out, int32_t* shares_out, int shares_cap);
int psmc_step_share_of(int R, int V, psmc_dtype dt, int granule);

/* Synchronises `stream` and returns the sticky device status word (PSMC_OK if
 * nothing went wrong since the last reset). */
psmc_status psmc_sync_status(psmc_ctx*, void* stream);
const char* psmc_strerror(psmc_status);

#ifdef __cplusplus
}
#endif
#endif /* PSMC_H */
