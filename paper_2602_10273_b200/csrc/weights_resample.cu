// Second kernel of the step: per-row finish of the logit pass, then weights, ESS and ESS-triggered
// systematic resampling (Algorithm 1 rows 5-16, Eq. 5, Eq. 7, and the stage-boundary update of
// Section 4.3 / Appendix B).  One CTA per group.
//
// Phase 1 (finish_rows: up to eight warps per particle, the CTA's warps shared among the group's rows):
// the span triples of the streaming kernel become the drawn token y, log p(y) and log omega of each row.
// Phase 2 (one thread per particle, N <= 1024); reductions and prefix sums run on warp shuffles plus a
// 33-entry shared array, in an order fixed by the thread index:
//   log W_r += (alpha_t - alpha_{t-1}) * S_r                     stage boundary (all rows)
//   live:  log W_r += log omega_r;  S_r += log p(y);  len_r += 1;  done_r |= (y == EOS)
//   done:  y = EOS, factor 1
//   w_i = exp(log W_i - max), C = inclusive prefix of w, ESS = (sum w)^2 / sum w^2.
//   If ESS < kappa*N:  u0 = hash uniform, A_i = min{j : C_j * N >= (u0 + i) * C_{N-1}} (N-1 if none),
//   offspring counts -> hazard-free slot map (survivors stay; dead slots, in increasing order, take
//   the surplus offspring, sources in increasing order), state gathered by the map, log W <- 0,
//   log Z-hat += max + log(sum w / N).  Move records for the KV reindex are appended to global lists.
#include "internal.h"
#include "logits_common.cuh"

namespace psmc {
namespace {

struct KernelArgs {
    WeightsArgs a;
    FinishParams f;
    int wpr;  // warps per row in the finish
};

template <int DT, int MODE>
__global__ void __launch_bounds__(1024) finish_weights_resample_kernel(const __grid_constant__ KernelArgs ka) {
    __shared__ double sh_red[33];
    __shared__ int sh_redi[33];
    __shared__ double sh_C[kMaxParticles];    // phase 1: log omega; phase 2: weight prefix
    __shared__ double sh_S[kMaxParticles];    // phase 1: log p(y);  phase 2: cumulative log p
    __shared__ int sh_off[kMaxParticles];
    __shared__ int sh_Einc[kMaxParticles];
    __shared__ int sh_len[kMaxParticles];
    __shared__ int sh_tok[kMaxParticles];
    __shared__ unsigned char sh_done[kMaxParticles];
    __shared__ int sh_base[2];
    __shared__ FinishShared sh_fin;

    const WeightsArgs& a = ka.a;
    const int g = blockIdx.x, i = threadIdx.x, N = a.N;

    chain_begin();
    // ---- phase 1: the CTA's warps finish the rows of the group's live particles ----
    finish_rows<DT, MODE>(
        ka.f, sh_fin, g * N, N, ka.wpr, [&](int k) { return a.done[g * N + k] == 0; },
        [&](int k) { return hash_uniform(hash5(a.seed, kStreamToken, (uint64_t)g, (uint64_t)a.t, (uint64_t)k)); },
        [&](int k, const RowResult& rr) {
            if (rr.tok < 0) raise_status(a.status, PSMC_E_NUMERIC);
            sh_tok[k] = rr.tok;
            sh_S[k] = rr.logp;
            sh_C[k] = rr.loginc;
        });
    // finish_rows ends on a CTA-wide barrier: the results are visible to every thread

    // ---- phase 2: per-particle update ----
    const int nw = (N + 31) >> 5;  // warps that hold particles
    if (nw == 1 && i >= 32) return;  // up to 32 particles: warp 0 finishes alone, on warp collectives only
    const bool on = i < N;
    const int r = g * N + (on ? i : 0);
    double lw = -INFINITY, S = 0.0;
    int tk = a.eos, ln = 0;
    unsigned char dn = 1;
    if (on) {
        dn = a.done[r];
        S = a.S[r];
        ln = a.len[r];
        lw = a.logW[r] + a.delta * S;
        double lp = 0.0, inc = 0.0;
        if (!dn) {
            tk = sh_tok[i];
            lp = sh_S[i];
            inc = sh_C[i];
            if (tk < 0) {  // the row was flagged: keep indices valid, leave the weight alone
                tk = a.eos;
                lp = 0.0;
                inc = 0.0;
            }
            lw += inc;
            S += lp;
            ln += 1;
            if (tk == a.eos) dn = 1;
        }
        a.logp[r] = lp;
        a.loginc[r] = inc;
        a.tok[r] = tk;
        a.hist_tok[r] = tk;
    }

    // ---- normalise, ESS (Eq. 5) ----
    const double M = block_max(lw, sh_red, nw);
    const double w = on ? exp(lw - M) : 0.0;
    double s1;
    const double C = block_scan_incl(w, sh_red, &s1, nw);
    const double s2 = block_sum(w * w, sh_red, nw);
    const double ess = s1 * s1 / s2;
    const bool fire = ess < a.kappa * (double)N;
    if (i == 0) {
        a.ess[g] = ess;
        a.resampled[g] = fire ? 1 : 0;
    }

    if (!fire) {
        if (on) {
            a.logW[r] = lw;
            a.S[r] = S;
            a.done[r] = dn;
            a.len[r] = ln;
            a.anc[r] = i;
            a.map[r] = i;
            a.hist_map[r] = i;
            a.last_tok[r] = tk;
        }
        return;
    }

    // ---- systematic resampling ----
    if (on) {
        sh_C[i] = C;
        sh_S[i] = S;
        sh_len[i] = ln;
        sh_tok[i] = tk;
        sh_done[i] = dn;
        sh_off[i] = 0;
    }
    group_sync(nw);
    int anc = N - 1;
    if (on) {
        const double u0 = hash_uniform(hash5(a.seed, kStreamResample, (uint64_t)g, (uint64_t)a.t, 0));
        const double pos = (u0 + (double)i) * s1;
        int lo = 0, hi = N;  // first j in [0,N) with C_j * N >= pos; C is non-decreasing
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (sh_C[mid] * (double)N >= pos) hi = mid; else lo = mid + 1;
        }
        anc = lo < N ? lo : N - 1;
        atomicAdd(&sh_off[anc], 1);
    }
    group_sync(nw);

    // ---- slot map ----
    const int off = on ? sh_off[i] : 1;
    const int dead = (on && off == 0) ? 1 : 0;
    const int surplus = (on && off > 1) ? off - 1 : 0;
    int n_dead, n_src;
    const int dead_incl = block_scan_incl(dead, sh_redi, &n_dead, nw);
    const int sur_incl = block_scan_incl(surplus, sh_redi, (int*)nullptr, nw);
    const int src_incl = block_scan_incl(surplus > 0 ? 1 : 0, sh_redi, &n_src, nw);
    if (on) sh_Einc[i] = sur_incl;
    if (i == 0) {
        sh_base[0] = atomicAdd(a.n_moves, n_dead);
        sh_base[1] = atomicAdd(a.n_sources, n_src);
    }
    group_sync(nw);
    int mp = i;
    if (dead) {
        const int rank = dead_incl - 1;  // this dead slot takes surplus offspring number `rank`
        int lo = 0, hi = N;              // first j with Einc[j] > rank
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (sh_Einc[mid] > rank) hi = mid; else lo = mid + 1;
        }
        mp = lo < N ? lo : N - 1;
        a.dst_rows[sh_base[0] + rank] = r;
    }
    if (surplus > 0) {
        MoveSource ms;
        ms.src_row = r;
        ms.len = ln;
        ms.dst_begin = sh_base[0] + (sur_incl - surplus);
        ms.n_dst = surplus;
        a.sources[sh_base[1] + src_incl - 1] = ms;
    }

    // ---- copy particle state by the map, uniform weights ----
    if (on) {
        a.logW[r] = 0.0;
        a.S[r] = sh_S[mp];
        a.done[r] = sh_done[mp];
        a.len[r] = sh_len[mp];
        a.anc[r] = anc;
        a.map[r] = mp;
        a.hist_map[r] = mp;
        a.last_tok[r] = sh_tok[mp];
    }
    if (i == 0) a.logZ[g] += M + log(s1 / (double)N);
}

typedef void (*Fn)(const KernelArgs);
template <int DT>
Fn pick(int mode) {
    switch (mode) {
        case kBeta1: return finish_weights_resample_kernel<DT, kBeta1>;
        case kBeta2: return finish_weights_resample_kernel<DT, kBeta2>;
        case kBeta4: return finish_weights_resample_kernel<DT, kBeta4>;
        case kBeta8: return finish_weights_resample_kernel<DT, kBeta8>;
        default: return finish_weights_resample_kernel<DT, kBetaAny>;
    }
}

}  // namespace

cudaError_t launch_weights_resample(const WeightsArgs& a, cudaStream_t stream) {
    const LogitsGeometry g = logits_geometry(a.logits, a.dt, a.R, a.V, a.ld, a.beta);
    KernelArgs ka;
    ka.a = a;
    ka.f.logits = a.logits; ka.f.V = a.V; ka.f.ld = a.ld; ka.f.span = g.span; ka.f.n_spans = g.n_spans;
    ka.f.partials = reinterpret_cast<const float4*>(a.scratch); ka.f.beta = a.beta; ka.f.alpha_t = a.alpha_t;
    ka.f.bf = g.bf; ka.f.vec = g.vec;
    // up to eight warps per particle while the CTA has room for them; beyond 32 particles the warps loop over rows
    const int wpr = finish_warps_per_row(a.N, g.span, kFinishMaxWarps);
    const int warps = a.N * wpr < kFinishMaxWarps ? a.N * wpr : kFinishMaxWarps;
    ka.wpr = wpr;
    Fn fn = a.dt == PSMC_F32 ? pick<PSMC_F32>(g.mode) : pick<PSMC_BF16>(g.mode);
    return launch_chained(fn, dim3((unsigned)a.G), dim3((unsigned)(warps * 32)), 0, stream, ka);
}

}  // namespace psmc
