// Context, argument checks and the extern "C" face of libpsmc.so.  The arithmetic of the step
// lives in the kernels; this file owns device state, computes the exponent schedule of
// Section 4.3 for the token at hand and enqueues the kernels on the caller's stream.
#include <map>
#include <mutex>
#include <new>
#include <utility>
#include <string.h>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "internal.h"

using namespace psmc;

namespace psmc {
cudaError_t allow_dynamic_smem(const void* kernel, int bytes) {
    static std::mutex mu;
    static std::map<std::pair<const void*, int>, int> granted;  // (kernel, device) -> bytes already allowed
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    int& have = granted[std::make_pair(kernel, dev)];
    if (have >= bytes) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) have = bytes;
    return e;
}
}  // namespace psmc

struct psmc_ctx {
    int device;
    int G, N, V, R, ramp, eos, T_max, t, resampler;
    double alpha, tau, kappa;
    uint64_t seed;
    int top_k;        // proposal restricted to the top of the row (masked_proposal.cu): at most one of the two is set
    double top_p;
    int32_t* set_size;  // [R] size of the proposal's support at the last step
    int32_t* prompt_len_host;  // [G]
    int32_t* prompt_len_dev;   // [G] the same on the device (for the shared-prompt form of the KV reindex)
    PagedState paged;          // block table, reference counts and free list of the paged cache (zero until created)
    // particle state
    double *logW, *S;
    uint8_t* done2[2];  // finished flags after steps of even / odd index: step t reads [(t-1)&1] and writes [t&1]
    int32_t* len;
    // results of the last step
    int32_t *tok, *last_tok, *anc, *map, *resampled;
    double *logp, *loginc, *ess, *logZ;
    // ancestry log for psmc_select
    int32_t *hist_tok, *hist_map;  // [T_max][R]
    // move records: [0] from the step, [1] from an idx_override
    MoveSource* sources[2];
    int32_t* dst_rows[2];
    int32_t* counts[3];  // {n_sources, n_moves}: [0]/[1] steps of even/odd index (they alternate), [2] idx_override
    int32_t* row_arrivals;    // [R] arrival counters of the one-kernel step (zero between launches)
    int32_t* group_arrivals;  // [G]
    void* step_triples;       // its triples of rows shared between CTAs
    int32_t* status;
    int32_t* kv_work;    // [2] unit queue of the reindex kernels (kept at zero between launches by the kernels)
    void* scratch;       // span triples of the logit pass
    size_t scratch_bytes;
    // the step with the vocabulary split over ranks: 0 = idle, 1 = swept, 2 = located; the local columns of the sweep
    int shard_phase, shard_P;
    LogitsStreamArgs shard_la;
    // the step fed one vocabulary tile at a time: 0 = idle, 1 = tiles coming in, 2 = owner columns handed out
    int tile_phase, tile_width, tiles_fed, tile_next_v0;
    double* tile_triples;          // [tile_cap][R][3]
    int tile_cap;
    psmc_shard_pick* tile_picks;   // [R]
    void* staging;       // psmc_step_host: device copy of the host logits
    size_t staging_bytes;
    cudaStream_t copy_stream;  // psmc_step_host: the logits travel on a stream of their own, so that the copy
    cudaEvent_t staged;        // overlaps whatever the caller still has running on its stream (the cache move)
    // optional per-kernel timing (psmc_timing_enable): event pairs recorded around every launch
    int timing_on;
    struct Timed { cudaEvent_t a, b; int kind; };
    std::vector<Timed> timed;
    std::vector<cudaEvent_t> event_pool;
};

namespace {

// A named range around the launches of one call, for timelines of tools that follow NVTX (header-only: without such a
// tool attached a push or pop is one test of a pointer).
struct TraceRange {
    explicit TraceRange(const char* name) { nvtxRangePushA(name); }
    ~TraceRange() { nvtxRangePop(); }
    TraceRange(const TraceRange&) = delete;
    TraceRange& operator=(const TraceRange&) = delete;
};

// finished flags after the steps taken so far
uint8_t* done_now(const psmc_ctx* c) { return c->done2[c->t & 1]; }

template <typename T>
cudaError_t dev_alloc(T** p, size_t count) {
    return cudaMalloc(reinterpret_cast<void**>(p), (count ? count : 1) * sizeof(T));
}

// Section 4.3 with one stage per token: alpha_t = 1 + (alpha - 1) * min(t, T_ramp) / T_ramp
double alpha_at(const psmc_ctx* c, int t) {
    if (c->ramp <= 0) return c->alpha;
    const int s = t < c->ramp ? t : c->ramp;
    return 1.0 + (c->alpha - 1.0) * (double)s / (double)c->ramp;
}

psmc_status reset_device_state(psmc_ctx* c) {
    const size_t R = (size_t)c->R, G = (size_t)c->G;
    cudaError_t e = cudaSuccess;
    auto z = [&](void* p, size_t bytes) { if (e == cudaSuccess) e = cudaMemset(p, 0, bytes); };
    z(c->logW, 8 * R); z(c->S, 8 * R); z(c->done2[0], R); z(c->done2[1], R);
    z(c->logp, 8 * R); z(c->loginc, 8 * R); z(c->logZ, 8 * G); z(c->resampled, 4 * G);
    z(c->counts[0], 8); z(c->counts[1], 8); z(c->counts[2], 8); z(c->status, 4); z(c->kv_work, 8);
    z(c->row_arrivals, 4 * R); z(c->group_arrivals, 4 * G); z(c->set_size, 4 * R);
    if (e != cudaSuccess) return PSMC_E_CUDA;
    // lens = prompt length of the group; identity maps; tokens -1; ESS = N
    int32_t* h = new (std::nothrow) int32_t[R];
    double* hd = new (std::nothrow) double[G];
    if (!h || !hd) { delete[] h; delete[] hd; return PSMC_E_NOMEM; }
    for (size_t r = 0; r < R; ++r) h[r] = c->prompt_len_host[r / c->N];
    e = cudaMemcpy(c->len, h, 4 * R, cudaMemcpyHostToDevice);
    for (size_t r = 0; r < R; ++r) h[r] = (int32_t)(r % c->N);
    if (e == cudaSuccess) e = cudaMemcpy(c->anc, h, 4 * R, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(c->map, h, 4 * R, cudaMemcpyHostToDevice);
    for (size_t r = 0; r < R; ++r) h[r] = -1;
    if (e == cudaSuccess) e = cudaMemcpy(c->tok, h, 4 * R, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(c->last_tok, h, 4 * R, cudaMemcpyHostToDevice);
    for (size_t g = 0; g < G; ++g) hd[g] = (double)c->N;
    if (e == cudaSuccess) e = cudaMemcpy(c->ess, hd, 8 * G, cudaMemcpyHostToDevice);
    delete[] h;
    delete[] hd;
    c->t = 0;
    c->shard_phase = 0;
    c->tile_phase = 0;
    return e == cudaSuccess ? PSMC_OK : PSMC_E_CUDA;
}

// Brackets one kernel launch with events on the caller's stream when timing is on.
struct LaunchTimer {
    psmc_ctx* c;
    cudaStream_t s;
    psmc_ctx::Timed t;
    bool on;
    // level: 1 = a single kernel, 2 = a whole call; the bracket is taken when it matches the mode that is switched on
    LaunchTimer(psmc_ctx* ctx, cudaStream_t stream, int kind, int level = 1)
        : c(ctx), s(stream), on(ctx->timing_on == level) {
        if (!on) return;
        cudaEvent_t ev[2];
        for (int i = 0; i < 2; ++i) {
            if (!c->event_pool.empty()) {
                ev[i] = c->event_pool.back();
                c->event_pool.pop_back();
            } else if (cudaEventCreate(&ev[i]) != cudaSuccess) {
                on = false;
                return;
            }
        }
        t.a = ev[0]; t.b = ev[1]; t.kind = kind;
        cudaEventRecord(t.a, s);
    }
    ~LaunchTimer() {
        if (!on) return;
        cudaEventRecord(t.b, s);
        c->timed.push_back(t);
    }
};

void free_ctx(psmc_ctx* c) {
    if (!c) return;
    for (auto& t : c->timed) { cudaEventDestroy(t.a); cudaEventDestroy(t.b); }
    for (auto e : c->event_pool) cudaEventDestroy(e);
    if (c->staged) cudaEventDestroy(c->staged);
    if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
    void* ptrs[] = {c->logW, c->S, c->done2[0], c->done2[1], c->len, c->tok, c->last_tok, c->anc, c->map, c->resampled,
                    c->logp, c->loginc, c->ess, c->logZ, c->hist_tok, c->hist_map, c->sources[0], c->sources[1],
                    c->dst_rows[0], c->dst_rows[1], c->counts[0], c->counts[1], c->counts[2], c->row_arrivals,
                    c->group_arrivals, c->step_triples, c->tile_triples, c->tile_picks, c->status, c->kv_work, c->scratch, c->staging, c->prompt_len_dev, c->set_size};
    for (void* p : ptrs)
        if (p) cudaFree(p);
    void* paged_ptrs[] = {c->paged.table, c->paged.refc, c->paged.free_list, c->paged.free_top};
    for (void* p : paged_ptrs)
        if (p) cudaFree(p);
    delete[] c->prompt_len_host;
    delete c;
}

}  // namespace

extern "C" psmc_status psmc_init_batched(psmc_ctx** out, int G, int N, int V, float alpha, float tau, float ess_thresh,
                                         int ramp, uint64_t seed, int eos_id, int T_max,
                                         const int32_t* prompt_len_host) {
    if (!out) return PSMC_E_INVAL;
    *out = nullptr;
    if (G < 1 || N < 1 || N > kMaxParticles || V < 2 || !(alpha >= 1.f) || !(tau > 0.f) || !(ess_thresh > 0.f) ||
        !(ess_thresh <= 1.f) || ramp < 0 || eos_id < 0 || eos_id >= V || T_max < 1)
        return PSMC_E_INVAL;
    if ((int64_t)G * N > (1 << 24)) return PSMC_E_INVAL;
    psmc_ctx* c = new (std::nothrow) psmc_ctx();
    if (!c) return PSMC_E_NOMEM;
    if (cudaGetDevice(&c->device) != cudaSuccess) { delete c; return PSMC_E_CUDA; }
    c->G = G; c->N = N; c->V = V; c->R = G * N; c->ramp = ramp; c->eos = eos_id; c->T_max = T_max;
    c->alpha = (double)alpha; c->tau = (double)tau; c->kappa = (double)ess_thresh; c->seed = seed;
    c->prompt_len_host = new (std::nothrow) int32_t[G];
    if (!c->prompt_len_host) { free_ctx(c); return PSMC_E_NOMEM; }
    for (int g = 0; g < G; ++g) {
        c->prompt_len_host[g] = prompt_len_host ? prompt_len_host[g] : 0;
        if (c->prompt_len_host[g] < 0) { free_ctx(c); return PSMC_E_INVAL; }
    }
    const size_t R = (size_t)c->R;
    cudaError_t e = cudaSuccess;
    auto ok = [&](cudaError_t x) { if (e == cudaSuccess) e = x; };
    ok(dev_alloc(&c->logW, R)); ok(dev_alloc(&c->S, R)); ok(dev_alloc(&c->done2[0], R)); ok(dev_alloc(&c->done2[1], R));
    ok(dev_alloc(&c->len, R));
    ok(dev_alloc(&c->tok, R)); ok(dev_alloc(&c->last_tok, R));
    ok(dev_alloc(&c->anc, R)); ok(dev_alloc(&c->map, R)); ok(dev_alloc(&c->resampled, (size_t)G));
    ok(dev_alloc(&c->logp, R)); ok(dev_alloc(&c->loginc, R)); ok(dev_alloc(&c->ess, (size_t)G));
    ok(dev_alloc(&c->set_size, R));
    ok(dev_alloc(&c->logZ, (size_t)G));
    ok(dev_alloc(&c->hist_tok, R * (size_t)T_max)); ok(dev_alloc(&c->hist_map, R * (size_t)T_max));
    for (int s = 0; s < 2; ++s) {
        ok(dev_alloc(&c->sources[s], R)); ok(dev_alloc(&c->dst_rows[s], R));
    }
    for (int s = 0; s < 3; ++s) ok(dev_alloc(&c->counts[s], 2));
    ok(dev_alloc(&c->row_arrivals, R)); ok(dev_alloc(&c->group_arrivals, (size_t)G));
    ok(cudaMalloc(&c->step_triples, step_fused_scratch_bytes()));
    ok(dev_alloc(&c->prompt_len_dev, (size_t)G));
    if (e == cudaSuccess) e = cudaMemcpy(c->prompt_len_dev, c->prompt_len_host, 4 * (size_t)G, cudaMemcpyHostToDevice);
    ok(dev_alloc(&c->status, 1));
    ok(dev_alloc(&c->kv_work, 2));
    c->scratch_bytes = logits_pass_scratch_bytes(c->R, c->V);
    ok(cudaMalloc(&c->scratch, c->scratch_bytes));
    if (e != cudaSuccess) { free_ctx(c); return e == cudaErrorMemoryAllocation ? PSMC_E_NOMEM : PSMC_E_CUDA; }
    psmc_status st = reset_device_state(c);
    if (st != PSMC_OK) { free_ctx(c); return st; }
    if (cudaDeviceSynchronize() != cudaSuccess) { free_ctx(c); return PSMC_E_CUDA; }
    *out = c;
    return PSMC_OK;
}

extern "C" psmc_status psmc_init(psmc_ctx** out, int N, int V, float alpha, float tau, float ess_thresh, int ramp,
                                 uint64_t seed, int eos_id) {
    return psmc_init_batched(out, 1, N, V, alpha, tau, ess_thresh, ramp, seed, eos_id, 4096, nullptr);
}

extern "C" psmc_status psmc_set_resampler(psmc_ctx* c, psmc_resampler kind) {
    if (!c || (int)kind < 0 || (int)kind > 3) return PSMC_E_INVAL;
    c->resampler = (int)kind;
    return PSMC_OK;
}

extern "C" psmc_status psmc_set_proposal_mask(psmc_ctx* c, int top_k, double top_p) {
    if (!c || top_k < 0 || !(top_p >= 0.0) || top_p > 1.0 || (top_k > 0 && top_p > 0.0)) return PSMC_E_INVAL;
    if (c->shard_phase != 0) return PSMC_E_STATE;
    c->top_k = top_k;
    c->top_p = top_p;
    return PSMC_OK;
}

extern "C" psmc_status psmc_destroy(psmc_ctx* c) {
    if (!c) return PSMC_E_INVAL;
    cudaDeviceSynchronize();
    free_ctx(c);
    return PSMC_OK;
}

extern "C" psmc_status psmc_reset(psmc_ctx* c, uint64_t seed) {
    TraceRange trace("psmc_reset");
    if (!c) return PSMC_E_INVAL;
    if (cudaDeviceSynchronize() != cudaSuccess) return PSMC_E_CUDA;
    c->seed = seed;
    psmc_status st = reset_device_state(c);
    if (st != PSMC_OK) return st;
    return cudaDeviceSynchronize() == cudaSuccess ? PSMC_OK : PSMC_E_CUDA;
}

namespace {

// The exponents of step t (Section 4.3 / Appendix B) and everything the per-group update reads and writes.
struct StepExponents {
    double alpha_t, alpha_prev, beta_t;
};
StepExponents exponents_at(const psmc_ctx* c, int t) {
    StepExponents x;
    x.alpha_t = alpha_at(c, t);
    x.alpha_prev = alpha_at(c, t - 1);
    x.beta_t = x.alpha_t / (c->alpha * c->tau);  // tau = 1/alpha gives beta_t = alpha_t (Corollary 1)
    return x;
}

// the span triples of a part of a row can take more room than those of the whole row (shorter spans)
psmc_status grow_scratch(psmc_ctx* c, size_t need, cudaStream_t s) {
    if (need <= c->scratch_bytes) return PSMC_OK;
    if (cudaStreamSynchronize(s) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) return PSMC_E_CUDA;
    cudaFree(c->scratch);
    c->scratch = nullptr;
    c->scratch_bytes = 0;
    if (cudaMalloc(&c->scratch, need) != cudaSuccess) return PSMC_E_NOMEM;
    c->scratch_bytes = need;
    return PSMC_OK;
}

WeightsArgs weights_args(psmc_ctx* c, int t, const StepExponents& x) {
    WeightsArgs wa{};
    wa.G = c->G; wa.N = c->N; wa.R = c->R; wa.t = t; wa.eos = c->eos; wa.resampler = c->resampler;
    wa.alpha_t = x.alpha_t; wa.beta = x.beta_t; wa.delta = x.alpha_t - x.alpha_prev; wa.kappa = c->kappa;
    wa.seed = c->seed;
    wa.logp = c->logp; wa.loginc = c->loginc;
    wa.logW = c->logW; wa.S = c->S; wa.done = c->done2[(t - 1) & 1]; wa.done_out = c->done2[t & 1]; wa.len = c->len;
    wa.tok = c->tok; wa.last_tok = c->last_tok; wa.anc = c->anc; wa.map = c->map;
    wa.resampled = c->resampled; wa.ess = c->ess; wa.logZ = c->logZ;
    wa.hist_tok = c->hist_tok + (size_t)(t - 1) * c->R;
    wa.hist_map = c->hist_map + (size_t)(t - 1) * c->R;
    wa.sources = c->sources[0]; wa.dst_rows = c->dst_rows[0];
    wa.n_sources = c->counts[t & 1]; wa.n_moves = c->counts[t & 1] + 1;
    wa.status = c->status;
    return wa;
}

}  // namespace

extern "C" psmc_status psmc_step(psmc_ctx* c, const void* logits, psmc_dtype dt, int64_t ld, void* stream) {
    TraceRange trace("psmc_step");
    if (!c || !logits || ld < c->V || (dt != PSMC_F32 && dt != PSMC_BF16)) return PSMC_E_INVAL;
    if (c->t >= c->T_max || c->shard_phase != 0 || c->tile_phase != 0) return PSMC_E_STATE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int t = c->t + 1;
    const StepExponents x = exponents_at(c, t);

    LogitsStreamArgs la{};
    la.logits = logits; la.dt = dt; la.R = c->R; la.V = c->V; la.ld = ld; la.beta = x.beta_t;
    la.done = done_now(c); la.scratch = c->scratch;
    la.status = c->status;
    la.zero_words = c->counts[(t + 1) & 1];  // each step clears the pair of move counters the next step will use

    WeightsArgs wa = weights_args(c, t, x);
    wa.logits = logits; wa.dt = dt; wa.V = c->V; wa.ld = ld; wa.scratch = c->scratch;
    LaunchTimer whole(c, s, 0, 2);
    if (c->top_k > 0 || c->top_p > 0.0) {  // proposal restricted to the top of the row: a pass of its own
        LaunchTimer lt(c, s, 0);
        if (launch_step_masked(la, wa, c->top_k, c->top_p, c->set_size, s) != cudaSuccess) return PSMC_E_CUDA;
    } else if (step_can_fuse(la, c->N)) {  // the whole step as one kernel
        LaunchTimer lt(c, s, 0);
        if (launch_step_fused(la, wa, c->step_triples, c->row_arrivals, c->group_arrivals, s) != cudaSuccess) return PSMC_E_CUDA;
    } else {
        {
            LaunchTimer lt(c, s, 0);
            if (launch_logits_stream(la, s) != cudaSuccess) return PSMC_E_CUDA;
        }
        LaunchTimer lt(c, s, 1);
        if (launch_weights_resample(wa, s) != cudaSuccess) return PSMC_E_CUDA;
    }
    c->t = t;
    return PSMC_OK;
}

// ---- the step with the vocabulary split over ranks (vocab_shard.cu) ----
extern "C" psmc_status psmc_shard_sweep(psmc_ctx* c, const void* logits_local, psmc_dtype dt, int64_t ld, int V_local,
                                        double* triples_out, void* stream) {
    TraceRange trace("psmc_shard_sweep");
    if (!c || !logits_local || !triples_out || V_local < 2 || V_local > c->V || ld < V_local ||
        (dt != PSMC_F32 && dt != PSMC_BF16))
        return PSMC_E_INVAL;
    if (c->t >= c->T_max || c->shard_phase != 0 || c->tile_phase != 0) return PSMC_E_STATE;
    if (c->top_k > 0 || c->top_p > 0.0) return PSMC_E_STATE;  // ranking a row needs all of its columns
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // a shard is cut into spans of its own; with many ranks that can take a few more triples than the whole row
    psmc_status grown = grow_scratch(c, logits_pass_scratch_bytes(c->R, V_local), s);
    if (grown != PSMC_OK) return grown;
    const int t = c->t + 1;
    const StepExponents x = exponents_at(c, t);
    LogitsStreamArgs la{};
    la.logits = logits_local; la.dt = dt; la.R = c->R; la.V = V_local; la.ld = ld; la.beta = x.beta_t;
    la.done = done_now(c); la.scratch = c->scratch;
    la.status = c->status;
    la.zero_words = c->counts[(t + 1) & 1];
    LaunchTimer lt(c, s, 0);
    if (launch_logits_stream(la, s) != cudaSuccess) return PSMC_E_CUDA;
    if (launch_shard_triples(la, triples_out, s) != cudaSuccess) return PSMC_E_CUDA;
    c->shard_la = la;
    c->shard_phase = 1;
    return PSMC_OK;
}

extern "C" psmc_status psmc_shard_locate(psmc_ctx* c, int v0, const double* all_triples, int P, int rank,
                                         psmc_shard_pick* picks_out, void* stream) {
    TraceRange trace("psmc_shard_locate");
    if (!c || !all_triples || !picks_out || P < 1 || P > 1024 || rank < 0 || rank >= P || v0 < 0) return PSMC_E_INVAL;
    if (c->shard_phase != 1) return PSMC_E_STATE;
    if ((int64_t)v0 + c->shard_la.V > c->V) return PSMC_E_INVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int t = c->t + 1;
    ShardLocateArgs sa{};
    sa.all_triples = all_triples; sa.P = P; sa.rank = rank; sa.N = c->N; sa.t = t; sa.v0 = v0;
    sa.alpha_t = alpha_at(c, t); sa.seed = c->seed; sa.picks_out = picks_out;
    LaunchTimer lt(c, s, 0);
    if (launch_shard_locate(c->shard_la, sa, s) != cudaSuccess) return PSMC_E_CUDA;
    c->shard_P = P;
    c->shard_phase = 2;
    return PSMC_OK;
}

extern "C" psmc_status psmc_shard_finish(psmc_ctx* c, const double* all_triples, const psmc_shard_pick* all_picks,
                                         int P, void* stream) {
    TraceRange trace("psmc_shard_finish");
    if (!c || !all_triples || !all_picks) return PSMC_E_INVAL;
    if (c->shard_phase != 2) return PSMC_E_STATE;
    if (P != c->shard_P) return PSMC_E_INVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int t = c->t + 1;
    const WeightsArgs wa = weights_args(c, t, exponents_at(c, t));
    LaunchTimer lt(c, s, 1);
    if (launch_shard_weights(wa, all_triples, all_picks, P, s) != cudaSuccess) return PSMC_E_CUDA;
    c->t = t;
    c->shard_phase = 0;
    return PSMC_OK;
}

// ---- the step fed one vocabulary tile at a time (the consumer side of an LM-head GEMM that never writes [R, V]) ----
extern "C" psmc_status psmc_tiles_feed(psmc_ctx* c, const void* tile_logits, psmc_dtype dt, int64_t ld, int v0, int width,
                                       void* stream) {
    TraceRange trace("psmc_tiles_feed");
    if (!c || !tile_logits || width < 2 || ld < width || v0 < 0 || (dt != PSMC_F32 && dt != PSMC_BF16)) return PSMC_E_INVAL;
    if (c->t >= c->T_max || c->shard_phase != 0 || c->tile_phase > 1) return PSMC_E_STATE;
    if (c->top_k > 0 || c->top_p > 0.0) return PSMC_E_STATE;  // ranking a row needs all of its columns
    if ((int64_t)v0 + width > c->V) return PSMC_E_INVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (c->tile_phase == 0) {  // first tile of the step: it fixes the tile width
        if (v0 != 0) return PSMC_E_STATE;
        const int cap = (c->V + width - 1) / width;
        if (cap > 1024) return PSMC_E_INVAL;
        if (cap > c->tile_cap) {
            if (cudaStreamSynchronize(s) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) return PSMC_E_CUDA;
            if (c->tile_triples) cudaFree(c->tile_triples);
            c->tile_triples = nullptr;
            c->tile_cap = 0;
            if (cudaMalloc(reinterpret_cast<void**>(&c->tile_triples), (size_t)cap * c->R * 3 * sizeof(double)) != cudaSuccess)
                return PSMC_E_NOMEM;
            c->tile_cap = cap;
        }
        if (!c->tile_picks && dev_alloc(&c->tile_picks, (size_t)c->R) != cudaSuccess) return PSMC_E_NOMEM;
        c->tile_width = width;
        c->tiles_fed = 0;
        c->tile_next_v0 = 0;
    } else {  // tiles come in vocabulary order, all of one width but possibly the last
        if (v0 != c->tile_next_v0) return PSMC_E_STATE;
        if (width != c->tile_width && !(width < c->tile_width && v0 + width == c->V)) return PSMC_E_INVAL;
    }
    psmc_status grown = grow_scratch(c, logits_pass_scratch_bytes(c->R, width), s);
    if (grown != PSMC_OK) return grown;
    const int t = c->t + 1;
    const StepExponents x = exponents_at(c, t);
    LogitsStreamArgs la{};
    la.logits = tile_logits; la.dt = dt; la.R = c->R; la.V = width; la.ld = ld; la.beta = x.beta_t;
    la.done = done_now(c); la.scratch = c->scratch;
    la.status = c->status;
    la.zero_words = c->counts[(t + 1) & 1];
    LaunchTimer lt(c, s, 0);
    if (launch_logits_stream(la, s) != cudaSuccess) return PSMC_E_CUDA;
    if (launch_shard_triples(la, c->tile_triples + (size_t)c->tiles_fed * c->R * 3, s) != cudaSuccess) return PSMC_E_CUDA;
    c->tiles_fed += 1;
    c->tile_next_v0 = v0 + width;
    c->tile_phase = 1;
    return PSMC_OK;
}

extern "C" psmc_status psmc_tiles_need(psmc_ctx* c, int32_t* first_column_out, void* stream) {
    TraceRange trace("psmc_tiles_need");
    if (!c || !first_column_out) return PSMC_E_INVAL;
    if (c->tile_phase != 1 || c->tile_next_v0 != c->V) return PSMC_E_STATE;  // the tiles have to cover the vocabulary
    const int t = c->t + 1;
    const StepExponents x = exponents_at(c, t);
    if (launch_shard_owner_columns(c->tile_triples, c->tiles_fed, c->R, c->N, t, x.beta_t, c->seed, done_now(c),
                                   c->tile_width, first_column_out, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return PSMC_E_CUDA;
    c->tile_phase = 2;
    return PSMC_OK;
}

extern "C" psmc_status psmc_tiles_finish(psmc_ctx* c, const void* row_tiles, psmc_dtype dt, int64_t ld, void* stream) {
    TraceRange trace("psmc_tiles_finish");
    if (!c || !row_tiles || (dt != PSMC_F32 && dt != PSMC_BF16)) return PSMC_E_INVAL;
    if (c->tile_phase != 2) return PSMC_E_STATE;
    if (ld < c->tile_width) return PSMC_E_INVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    psmc_status grown = grow_scratch(c, logits_pass_scratch_bytes(c->R, c->tile_width), s);
    if (grown != PSMC_OK) return grown;
    const int t = c->t + 1;
    const StepExponents x = exponents_at(c, t);
    LogitsStreamArgs la{};
    la.logits = row_tiles; la.dt = dt; la.R = c->R; la.V = c->tile_width; la.ld = ld; la.beta = x.beta_t;
    la.done = done_now(c); la.scratch = c->scratch;
    la.status = c->status;
    la.zero_words = nullptr;
    ShardLocateArgs sa{};
    sa.all_triples = c->tile_triples; sa.P = c->tiles_fed; sa.rank = -1; sa.N = c->N; sa.t = t; sa.v0 = 0;
    sa.tile_width = c->tile_width; sa.alpha_t = x.alpha_t; sa.seed = c->seed; sa.picks_out = c->tile_picks;
    {
        LaunchTimer lt(c, s, 0);
        if (launch_logits_stream(la, s) != cudaSuccess) return PSMC_E_CUDA;
        if (launch_shard_locate(la, sa, s) != cudaSuccess) return PSMC_E_CUDA;
    }
    const WeightsArgs wa = weights_args(c, t, x);
    LaunchTimer lt(c, s, 1);
    if (launch_shard_weights(wa, c->tile_triples, c->tile_picks, c->tiles_fed, s, true) != cudaSuccess) return PSMC_E_CUDA;
    c->t = t;
    c->tile_phase = 0;
    return PSMC_OK;
}

extern "C" psmc_status psmc_step_host(psmc_ctx* c, const void* logits_host, psmc_dtype dt, int64_t ld,
                                      int32_t* tokens_out_host, void* stream) {
    TraceRange trace("psmc_step_host");
    if (!c || !logits_host || !tokens_out_host || ld < c->V || (dt != PSMC_F32 && dt != PSMC_BF16))
        return PSMC_E_INVAL;
    if (c->t >= c->T_max) return PSMC_E_STATE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t esize = dt == PSMC_F32 ? 4 : 2;
    // staging rows are padded to 16 bytes so that the 128-bit load path applies
    const int64_t ld_dev = ((int64_t)c->V * esize + 15) / 16 * 16 / esize;
    const size_t need = (size_t)c->R * ld_dev * esize;
    if (c->staging_bytes < need) {
        if (c->staging) { cudaStreamSynchronize(s); cudaFree(c->staging); c->staging = nullptr; c->staging_bytes = 0; }
        if (cudaMalloc(&c->staging, need) != cudaSuccess) return PSMC_E_NOMEM;
        c->staging_bytes = need;
    }
    // The staging buffer is free here: the previous call returned after its step had consumed it.  Work the caller
    // queued since (the cache move of the previous token) keeps running while the new logits come in.
    if (!c->copy_stream) {
        if (cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) != cudaSuccess) return PSMC_E_CUDA;
        if (cudaEventCreateWithFlags(&c->staged, cudaEventDisableTiming) != cudaSuccess) return PSMC_E_CUDA;
    }
    // one flat copy when both sides are dense (the usual case), row by row otherwise
    const cudaError_t copied =
        (ld == c->V && ld_dev == c->V)
            ? cudaMemcpyAsync(c->staging, logits_host, need, cudaMemcpyHostToDevice, c->copy_stream)
            : cudaMemcpy2DAsync(c->staging, ld_dev * esize, logits_host, ld * esize, (size_t)c->V * esize, c->R,
                                cudaMemcpyHostToDevice, c->copy_stream);
    if (copied != cudaSuccess ||
        cudaEventRecord(c->staged, c->copy_stream) != cudaSuccess || cudaStreamWaitEvent(s, c->staged, 0) != cudaSuccess)
        return PSMC_E_CUDA;
    psmc_status st = psmc_step(c, c->staging, dt, ld_dev, stream);
    if (st != PSMC_OK) return st;
    if (cudaMemcpyAsync(tokens_out_host, c->last_tok, 4 * (size_t)c->R, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return PSMC_E_CUDA;
    return cudaStreamSynchronize(s) == cudaSuccess ? PSMC_OK : PSMC_E_CUDA;
}

extern "C" psmc_status psmc_reindex_kv(psmc_ctx* c, const psmc_kv_desc* src, const psmc_kv_desc* dst,
                                       const int32_t* idx_override, void* stream) {
    TraceRange trace("psmc_reindex_kv");
    if (!c || !src || !src->k || !src->v) return PSMC_E_INVAL;
    if (src->n_layers < 1 || src->n_kv_heads < 1 || src->head_dim < 1 || src->max_len < 1) return PSMC_E_INVAL;
    if (src->dt != PSMC_F32 && src->dt != PSMC_BF16) return PSMC_E_INVAL;
    const int64_t min_head = (int64_t)src->max_len * src->head_dim;
    if (src->stride_head < min_head || src->stride_row < (int64_t)src->n_kv_heads * src->stride_head)
        return PSMC_E_INVAL;
    if (dst) {
        if (!dst->k || !dst->v || !idx_override) return PSMC_E_INVAL;  // out of place needs an explicit gather vector
        if (dst->n_layers != src->n_layers || dst->n_kv_heads != src->n_kv_heads || dst->head_dim != src->head_dim ||
            dst->max_len != src->max_len || dst->dt != src->dt)
            return PSMC_E_INVAL;
        if (dst->stride_head < min_head || dst->stride_row < (int64_t)dst->n_kv_heads * dst->stride_head)
            return PSMC_E_INVAL;
    }
    // the copy kernels number their work units in an int
    const int ptrs_per_launch = 2 * (src->n_layers < kMaxKvPtrs / 2 ? src->n_layers : kMaxKvPtrs / 2);
    if ((int64_t)c->R * ptrs_per_launch * src->n_kv_heads * reindex_unit_parts() >= ((int64_t)1 << 31)) return PSMC_E_INVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int set = idx_override ? 1 : 0;
    if (idx_override) {
        if (launch_build_moves(idx_override, c->R, src->max_len, dst ? 0 : 1, c->sources[1], c->dst_rows[1],
                               c->counts[2], c->counts[2] + 1, c->status, s) != cudaSuccess)
            return PSMC_E_CUDA;
    }
    const psmc_kv_desc* d = dst ? dst : src;
    const int64_t esize = src->dt == PSMC_F32 ? 4 : 2;
    KvLaunch k;
    k.H = src->n_kv_heads;
    k.row_bytes_stride = src->stride_row * esize;
    k.head_bytes_stride = src->stride_head * esize;
    k.dst_row_bytes_stride = d->stride_row * esize;
    k.dst_head_bytes_stride = d->stride_head * esize;
    k.pos_bytes = (int)(src->head_dim * esize);
    k.max_len = src->max_len;
    k.sources = c->sources[set];
    k.dst_rows = c->dst_rows[set];
    k.n_sources = idx_override ? c->counts[2] : c->counts[c->t & 1];
    k.status = c->status;
    k.work = c->kv_work;
    k.skip_pos = (!idx_override && src->skip_shared_prompt) ? c->prompt_len_dev : nullptr;
    k.N = c->N;
    uint64_t bits = (uint64_t)k.row_bytes_stride | (uint64_t)k.head_bytes_stride | (uint64_t)k.dst_row_bytes_stride |
                    (uint64_t)k.dst_head_bytes_stride | (uint64_t)k.pos_bytes;
    for (int l = 0; l < src->n_layers; ++l) {
        if (!src->k[l] || !src->v[l] || !d->k[l] || !d->v[l]) return PSMC_E_INVAL;
        bits |= (uint64_t)(uintptr_t)src->k[l] | (uint64_t)(uintptr_t)src->v[l] | (uint64_t)(uintptr_t)d->k[l] |
                (uint64_t)(uintptr_t)d->v[l];
    }
    k.bulk_ok = (bits % 16 == 0) ? 1 : 0;
    for (int l0 = 0; l0 < src->n_layers; l0 += kMaxKvPtrs / 2) {
        const int nl = src->n_layers - l0 < kMaxKvPtrs / 2 ? src->n_layers - l0 : kMaxKvPtrs / 2;
        for (int l = 0; l < nl; ++l) {
            k.src[2 * l] = static_cast<char*>(src->k[l0 + l]);
            k.src[2 * l + 1] = static_cast<char*>(src->v[l0 + l]);
            k.dst[2 * l] = static_cast<char*>(d->k[l0 + l]);
            k.dst[2 * l + 1] = static_cast<char*>(d->v[l0 + l]);
        }
        k.n_ptrs = 2 * nl;
        LaunchTimer lt(c, s, 2, c->timing_on ? c->timing_on : 1);  // bracketed in either mode
        if (launch_reindex_kv(k, s) != cudaSuccess) return PSMC_E_CUDA;
    }
    return PSMC_OK;
}

extern "C" psmc_status psmc_kv_paged_create(psmc_ctx* c, int n_blocks, int block_len, int max_blocks_per_row,
                                            int share_prompt) {
    if (!c || n_blocks < 1 || block_len < 1 || max_blocks_per_row < 1) return PSMC_E_INVAL;
    if (cudaDeviceSynchronize() != cudaSuccess) return PSMC_E_CUDA;
    PagedState& ps = c->paged;
    void* old[] = {ps.table, ps.refc, ps.free_list, ps.free_top};
    for (void* p : old)
        if (p) cudaFree(p);
    ps = PagedState{};
    ps.n_blocks = n_blocks; ps.block_len = block_len; ps.max_blocks = max_blocks_per_row; ps.R = c->R; ps.N = c->N;
    cudaError_t e = cudaSuccess;
    auto ok = [&](cudaError_t x) { if (e == cudaSuccess) e = x; };
    ok(dev_alloc(&ps.table, (size_t)c->R * max_blocks_per_row));
    ok(dev_alloc(&ps.refc, (size_t)n_blocks));
    ok(dev_alloc(&ps.free_list, paged_free_list_words(n_blocks, c->R)));
    ok(dev_alloc(&ps.free_top, 1));
    if (e != cudaSuccess) return e == cudaErrorMemoryAllocation ? PSMC_E_NOMEM : PSMC_E_CUDA;
    if (launch_paged_init(ps, c->prompt_len_dev, c->G, share_prompt, c->status, nullptr) != cudaSuccess) return PSMC_E_CUDA;
    return cudaDeviceSynchronize() == cudaSuccess ? PSMC_OK : PSMC_E_CUDA;
}

extern "C" psmc_status psmc_kv_paged_append(psmc_ctx* c, void* stream) {
    TraceRange trace("psmc_kv_paged_append");
    if (!c) return PSMC_E_INVAL;
    if (!c->paged.table) return PSMC_E_STATE;
    return launch_paged_append(c->paged, c->len, done_now(c), c->status, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? PSMC_OK : PSMC_E_CUDA;
}

extern "C" psmc_status psmc_reindex_kv_paged(psmc_ctx* c, const psmc_kv_pools* pools, void* stream) {
    TraceRange trace("psmc_reindex_kv_paged");
    if (!c || !pools || !pools->k || !pools->v) return PSMC_E_INVAL;
    if (!c->paged.table) return PSMC_E_STATE;
    if (pools->n_layers < 1 || pools->n_layers > kMaxKvPtrs / 2 || pools->n_kv_heads < 1 || pools->head_dim < 1)
        return PSMC_E_INVAL;
    if (pools->dt != PSMC_F32 && pools->dt != PSMC_BF16) return PSMC_E_INVAL;
    PagedPools pp;
    pp.n_layers = pools->n_layers; pp.H = pools->n_kv_heads;
    pp.pos_bytes = pools->head_dim * (pools->dt == PSMC_F32 ? 4 : 2);
    uint64_t bits = (uint64_t)pp.pos_bytes;
    for (int l = 0; l < pools->n_layers; ++l) {
        if (!pools->k[l] || !pools->v[l]) return PSMC_E_INVAL;
        pp.k[l] = static_cast<char*>(pools->k[l]);
        pp.v[l] = static_cast<char*>(pools->v[l]);
        bits |= (uint64_t)(uintptr_t)pools->k[l] | (uint64_t)(uintptr_t)pools->v[l];
    }
    if (bits % 16 != 0) return PSMC_E_INVAL;  // the block copy moves 16 bytes at a time
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    LaunchTimer lt(c, s, 2, c->timing_on ? c->timing_on : 1);
    // unless this was the last step the context can take, the rows are also made ready for the next token
    const bool more = c->t < c->T_max;
    return launch_paged_reindex(c->paged, pp, c->sources[0], c->dst_rows[0], c->counts[c->t & 1], c->counts[c->t & 1] + 1,
                                more ? c->len : nullptr, more ? done_now(c) : nullptr, c->status, s) == cudaSuccess
               ? PSMC_OK : PSMC_E_CUDA;
}

extern "C" const int32_t* psmc_kv_paged_table(psmc_ctx* c) { return c ? c->paged.table : nullptr; }
extern "C" const int32_t* psmc_kv_paged_refcount(psmc_ctx* c) { return c ? c->paged.refc : nullptr; }
extern "C" const int32_t* psmc_kv_paged_free_count(psmc_ctx* c) { return c ? c->paged.free_top : nullptr; }

extern "C" psmc_status psmc_select(psmc_ctx* c, int32_t* out_tokens, int32_t* out_len, int32_t* out_index,
                                   void* stream) {
    TraceRange trace("psmc_select");
    if (!c) return PSMC_E_INVAL;
    SelectArgs a{};
    a.G = c->G; a.N = c->N; a.R = c->R; a.t = c->t; a.T_max = c->T_max; a.eos = c->eos; a.seed = c->seed;
    a.logW = c->logW; a.hist_tok = c->hist_tok; a.hist_map = c->hist_map;
    a.out_tokens = out_tokens; a.out_len = out_len; a.out_index = out_index;
    return launch_select(a, static_cast<cudaStream_t>(stream)) == cudaSuccess ? PSMC_OK : PSMC_E_CUDA;
}

extern "C" psmc_status psmc_set_state(psmc_ctx* c, const double* log_w, const double* cum_logp, const uint8_t* done,
                                      const int32_t* lens) {
    if (!c) return PSMC_E_INVAL;
    if (cudaDeviceSynchronize() != cudaSuccess) return PSMC_E_CUDA;
    const size_t R = (size_t)c->R;
    cudaError_t e = cudaSuccess;
    if (log_w) e = cudaMemcpy(c->logW, log_w, 8 * R, cudaMemcpyHostToDevice);
    if (e == cudaSuccess && cum_logp) e = cudaMemcpy(c->S, cum_logp, 8 * R, cudaMemcpyHostToDevice);
    if (e == cudaSuccess && done) e = cudaMemcpy(done_now(c), done, R, cudaMemcpyHostToDevice);
    if (e == cudaSuccess && lens) e = cudaMemcpy(c->len, lens, 4 * R, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    return e == cudaSuccess ? PSMC_OK : PSMC_E_CUDA;
}

namespace {

struct SnapshotHeader {
    uint64_t magic;
    int32_t G, N, V, T_max, t, ramp, eos, resampler;
    double alpha, tau, kappa;
    uint64_t seed;
    double top_p;
    int32_t top_k, reserved;
};
constexpr uint64_t kSnapshotMagic = 0x33434d5350ull;  // "PSMC3"

// the device arrays of a snapshot, in file order; hist arrays only up to step t
struct Piece {
    void* dev;
    size_t bytes;
};
int snapshot_pieces(psmc_ctx* c, int t, Piece* out) {
    const size_t R = (size_t)c->R, G = (size_t)c->G;
    int n = 0;
    auto add = [&](void* p, size_t b) { out[n].dev = p; out[n].bytes = b; ++n; };
    add(c->logW, 8 * R); add(c->S, 8 * R); add(c->logp, 8 * R); add(c->loginc, 8 * R);
    add(c->ess, 8 * G); add(c->logZ, 8 * G);
    add(c->len, 4 * R); add(c->tok, 4 * R); add(c->last_tok, 4 * R); add(c->anc, 4 * R); add(c->map, 4 * R);
    add(c->resampled, 4 * G); add(c->status, 4);
    add(c->hist_tok, 4 * R * (size_t)t); add(c->hist_map, 4 * R * (size_t)t);
    add(c->done2[t & 1], R);
    return n;
}
size_t snapshot_bytes(psmc_ctx* c, int t) {
    Piece ps[20];
    const int n = snapshot_pieces(c, t, ps);
    size_t total = sizeof(SnapshotHeader) + 4 * (size_t)c->G;  // header, the G prompt lengths, the device arrays
    for (int i = 0; i < n; ++i) total += ps[i].bytes;
    return total;
}

}  // namespace

extern "C" size_t psmc_state_bytes(const psmc_ctx* c) {
    return c ? snapshot_bytes(const_cast<psmc_ctx*>(c), c->t) : 0;
}

extern "C" psmc_status psmc_state_save(psmc_ctx* c, void* host_buf, size_t bytes) {
    if (!c || !host_buf || bytes < snapshot_bytes(c, c->t)) return PSMC_E_INVAL;
    if (c->shard_phase != 0 || c->tile_phase != 0) return PSMC_E_STATE;  // inside a step there is no consistent state
    if (cudaDeviceSynchronize() != cudaSuccess) return PSMC_E_CUDA;
    SnapshotHeader h{};
    h.magic = kSnapshotMagic;
    h.G = c->G; h.N = c->N; h.V = c->V; h.T_max = c->T_max; h.t = c->t; h.ramp = c->ramp; h.eos = c->eos;
    h.resampler = c->resampler; h.alpha = c->alpha; h.tau = c->tau; h.kappa = c->kappa; h.seed = c->seed;
    h.top_k = c->top_k; h.top_p = c->top_p;
    char* out = static_cast<char*>(host_buf);
    memcpy(out, &h, sizeof(h));
    out += sizeof(h);
    memcpy(out, c->prompt_len_host, 4 * (size_t)c->G);
    out += 4 * (size_t)c->G;
    Piece ps[20];
    const int n = snapshot_pieces(c, c->t, ps);
    for (int i = 0; i < n; ++i) {
        if (ps[i].bytes && cudaMemcpy(out, ps[i].dev, ps[i].bytes, cudaMemcpyDeviceToHost) != cudaSuccess) return PSMC_E_CUDA;
        out += ps[i].bytes;
    }
    return PSMC_OK;
}

extern "C" psmc_status psmc_state_load(psmc_ctx* c, const void* host_buf, size_t bytes) {
    if (!c || !host_buf || bytes < sizeof(SnapshotHeader)) return PSMC_E_INVAL;
    SnapshotHeader h;
    memcpy(&h, host_buf, sizeof(h));
    if (h.magic != kSnapshotMagic || h.G != c->G || h.N != c->N || h.V != c->V || h.T_max != c->T_max || h.t < 0 ||
        h.t > c->T_max || h.resampler < 0 || h.resampler > 3)
        return PSMC_E_INVAL;
    if (bytes < snapshot_bytes(c, h.t)) return PSMC_E_INVAL;
    // the prompt lengths decide which cache positions the shared-prompt reindex and the paged cache leave alone:
    // a context created with other lengths would go on silently with the wrong ones
    if (memcmp(static_cast<const char*>(host_buf) + sizeof(h), c->prompt_len_host, 4 * (size_t)c->G) != 0) return PSMC_E_INVAL;
    if (cudaDeviceSynchronize() != cudaSuccess) return PSMC_E_CUDA;
    psmc_status st = reset_device_state(c);  // counters, arrival words and the rest of the scratch state start clean
    if (st != PSMC_OK) return st;
    const char* in = static_cast<const char*>(host_buf) + sizeof(h) + 4 * (size_t)c->G;
    Piece ps[20];
    const int n = snapshot_pieces(c, h.t, ps);
    for (int i = 0; i < n; ++i) {
        if (ps[i].bytes && cudaMemcpy(ps[i].dev, in, ps[i].bytes, cudaMemcpyHostToDevice) != cudaSuccess) return PSMC_E_CUDA;
        in += ps[i].bytes;
    }
    c->t = h.t; c->ramp = h.ramp; c->eos = h.eos; c->resampler = h.resampler;
    c->top_k = h.top_k; c->top_p = h.top_p;
    c->shard_phase = 0;
    c->alpha = h.alpha; c->tau = h.tau; c->kappa = h.kappa; c->seed = h.seed;
    return cudaDeviceSynchronize() == cudaSuccess ? PSMC_OK : PSMC_E_CUDA;
}

extern "C" psmc_status psmc_sync_status(psmc_ctx* c, void* stream) {
    if (!c) return PSMC_E_INVAL;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return PSMC_E_CUDA;
    int32_t w = 0;
    if (cudaMemcpy(&w, c->status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return PSMC_E_CUDA;
    return (psmc_status)w;
}

extern "C" psmc_status psmc_timing_enable(psmc_ctx* c, int on) {
    if (!c) return PSMC_E_INVAL;
    c->timing_on = on == 2 ? 2 : (on ? 1 : 0);
    return PSMC_OK;
}

extern "C" psmc_status psmc_timing_read(psmc_ctx* c, double* ms_out, int64_t* launches_out) {
    if (!c || !ms_out || !launches_out) return PSMC_E_INVAL;
    for (int k = 0; k < 3; ++k) { ms_out[k] = 0.0; launches_out[k] = 0; }
    psmc_status st = PSMC_OK;
    for (auto& t : c->timed) {
        float ms = 0.f;
        if (cudaEventSynchronize(t.b) != cudaSuccess || cudaEventElapsedTime(&ms, t.a, t.b) != cudaSuccess)
            st = PSMC_E_CUDA;
        if (t.kind >= 0 && t.kind < 3) { ms_out[t.kind] += (double)ms; launches_out[t.kind] += 1; }
        c->event_pool.push_back(t.a);
        c->event_pool.push_back(t.b);
    }
    c->timed.clear();
    return st;
}

extern "C" const char* psmc_strerror(psmc_status s) {
    switch (s) {
        case PSMC_OK: return "ok";
        case PSMC_E_INVAL: return "invalid argument";
        case PSMC_E_NOMEM: return "out of memory";
        case PSMC_E_CUDA: return "CUDA runtime error";
        case PSMC_E_STATE: return "call out of order";
        case PSMC_E_NUMERIC: return "NaN/+inf logit or a row without finite logits";
        case PSMC_E_TIMEOUT: return "bounded device wait ran out";
        case PSMC_E_HAZARD: return "in-place gather vector reads a row that is also written";
        case PSMC_E_TOO_LARGE: return "problem needs more than the fixed scratch of psmc_logits_pass_static";
    }
    return "unknown status";
}

extern "C" const int32_t* psmc_tokens(psmc_ctx* c) { return c ? c->tok : nullptr; }
extern "C" const int32_t* psmc_last_tokens(psmc_ctx* c) { return c ? c->last_tok : nullptr; }
extern "C" const double* psmc_log_weights(psmc_ctx* c) { return c ? c->logW : nullptr; }
extern "C" const double* psmc_log_inc(psmc_ctx* c) { return c ? c->loginc : nullptr; }
extern "C" const double* psmc_logp_tok(psmc_ctx* c) { return c ? c->logp : nullptr; }
extern "C" const double* psmc_cum_logp(psmc_ctx* c) { return c ? c->S : nullptr; }
extern "C" const int32_t* psmc_ancestors(psmc_ctx* c) { return c ? c->anc : nullptr; }
extern "C" const int32_t* psmc_slot_map(psmc_ctx* c) { return c ? c->map : nullptr; }
extern "C" const int32_t* psmc_resampled(psmc_ctx* c) { return c ? c->resampled : nullptr; }
extern "C" const double* psmc_ess(psmc_ctx* c) { return c ? c->ess : nullptr; }
extern "C" const double* psmc_log_z(psmc_ctx* c) { return c ? c->logZ : nullptr; }
extern "C" const int32_t* psmc_mask_sizes(psmc_ctx* c) { return c ? c->set_size : nullptr; }
extern "C" const int32_t* psmc_lens(psmc_ctx* c) { return c ? c->len : nullptr; }
extern "C" const uint8_t* psmc_done(psmc_ctx* c) { return c ? done_now(c) : nullptr; }
extern "C" const int32_t* psmc_move_count(psmc_ctx* c) { return c ? c->counts[c->t & 1] + 1 : nullptr; }
extern "C" int psmc_step_index(const psmc_ctx* c) { return c ? c->t : -1; }
extern "C" int psmc_rows(const psmc_ctx* c) { return c ? c->R : -1; }
