// Per-group part of the step (Algorithm 1: the per-particle updates, normalisation, trigger and resampling of its loop body): weight update with the stage-boundary term of Section 4.3 /
// Appendix B, absorbing EOS (Appendix D), normalisation and ESS (Eq. 5), the trigger ESS < kappa N, systematic
// resampling, the hazard-free slot map, the gather of the particle state by that map and the move records for the
// KV reindex.  One thread per particle; a team of `nw` warps (the first threads of a CTA, or one warp on its own
// when N <= 32).  Reductions and prefix sums run in an order fixed by the thread index.
//
//   log W_r += (alpha_t - alpha_{t-1}) * S_r                     stage boundary (all rows)
//   live:  log W_r += log omega_r;  S_r += log p(y);  len_r += 1;  done_r |= (y == EOS)
//   done:  y = EOS, factor 1
//   w_i = exp(log W_i - max), C = inclusive prefix of w, ESS = (sum w)^2 / sum w^2.
//   If ESS < kappa*N:  u0 = hash uniform, A_i = min{j : C_j * N >= (u0 + i) * C_{N-1}} (N-1 if none)
//   [systematic, the scheme of Algorithm 1; stratified, multinomial and residual resampling of Appendix E on request],
//   offspring counts -> slot map (survivors stay; dead slots, in increasing order, take the surplus offspring,
//   sources in increasing order), state gathered by the map, log W <- 0, log Z-hat += max + log(sum w / N).
#pragma once

#include "common.cuh"
#include "internal.h"

namespace psmc {

template <int CAP>
struct GroupScratch {
    double red[33];
    int redi[33];
    double C[CAP];  // weight prefix
    double S[CAP];  // cumulative log p
    double Rp[CAP];  // residual scheme: prefix of the residual weights
    int off[CAP];
    int Einc[CAP];
    int len[CAP];
    int tok[CAP];
    unsigned char done[CAP];
    int base[2];
};

// A particle's state as the step finds it; a kernel can fetch it early, while the row finishes are still running.
struct ParticleState {
    double logW, S;
    int len;
    unsigned char done;
};
__device__ __forceinline__ ParticleState load_particle(const WeightsArgs& a, int r) {
    ParticleState s;
    s.done = a.done[r];
    s.S = a.S[r];
    s.len = a.len[r];
    s.logW = a.logW[r];
    return s;
}

// i: this thread's index in the team (particle i when i < N).  tk_in / lp_in / inc_in: the row's drawn token
// (-1 when the row was flagged), log p(y) and log omega; ignored for finished rows.  st: the particle's state.
template <class Scratch>
__device__ __forceinline__ void group_update(const WeightsArgs& a, int g, int i, int nw, Scratch& sc, int tk_in, double lp_in,
                                             double inc_in, const ParticleState& st) {
    const int N = a.N;
    const bool on = i < N;
    const int r = g * N + (on ? i : 0);
    double lw = -INFINITY, S = 0.0;
    int tk = a.eos, ln = 0;
    unsigned char dn = 1;
    if (on) {
        dn = st.done;
        S = st.S;
        ln = st.len;
        lw = st.logW + a.delta * S;
        double lp = 0.0, inc = 0.0;
        if (!dn) {
            tk = tk_in;
            lp = lp_in;
            inc = inc_in;
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
    const double M = block_max(lw, sc.red, nw);
    const double w = on ? exp(lw - M) : 0.0;
    double s1;
    const double C = block_scan_incl(w, sc.red, &s1, nw);
    const double s2 = block_sum(w * w, sc.red, nw);
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
            a.done_out[r] = dn;
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
        sc.C[i] = C;
        sc.S[i] = S;
        sc.len[i] = ln;
        sc.tok[i] = tk;
        sc.done[i] = dn;
        sc.off[i] = 0;
    }
    group_sync(nw);
    int anc = N - 1;
    if (a.resampler == PSMC_RESAMPLE_RESIDUAL) {
        // floor(N W_j) copies of every j in order of j, the rest drawn from the residual weights (Appendix E)
        const double x = on ? (double)N * w / s1 : 0.0;
        const double fl = floor(x);
        int D;
        double res_total;
        const int d_incl = block_scan_incl(on ? (int)fl : 0, sc.redi, &D, nw);
        const double r_incl = block_scan_incl(on ? x - fl : 0.0, sc.red, &res_total, nw);
        if (on) {
            sc.Einc[i] = d_incl;
            sc.Rp[i] = r_incl;
        }
        group_sync(nw);
        if (on) {
            int lo = 0, hi = N;
            if (i < D) {  // first j whose copies reach beyond position i
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    if (sc.Einc[mid] > i) hi = mid; else lo = mid + 1;
                }
            } else {      // residual draw number i - D
                const double level =
                    hash_uniform(hash5(a.seed, kStreamResample, (uint64_t)g, (uint64_t)a.t, (uint64_t)(1 + i - D))) * res_total;
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    if (sc.Rp[mid] >= level) hi = mid; else lo = mid + 1;
                }
            }
            anc = lo < N ? lo : N - 1;
            atomicAdd(&sc.off[anc], 1);
        }
        group_sync(nw);  // Einc is written again below
    } else if (on) {
        // position of this particle against the weight prefix: first j with C_j * N >= pos (systematic, stratified)
        // or C_j >= level (multinomial); C is non-decreasing
        const bool multinomial = a.resampler == PSMC_RESAMPLE_MULTINOMIAL;
        const uint64_t which = a.resampler == PSMC_RESAMPLE_SYSTEMATIC ? 0 : (uint64_t)(1 + i);
        const double u = hash_uniform(hash5(a.seed, kStreamResample, (uint64_t)g, (uint64_t)a.t, which));
        const double pos = multinomial ? u * s1 : (u + (double)i) * s1;
        const double scale = multinomial ? 1.0 : (double)N;
        int lo = 0, hi = N;
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (sc.C[mid] * scale >= pos) hi = mid; else lo = mid + 1;
        }
        anc = lo < N ? lo : N - 1;
        atomicAdd(&sc.off[anc], 1);
    }
    group_sync(nw);

    // ---- slot map ----
    const int off = on ? sc.off[i] : 1;
    const int dead = (on && off == 0) ? 1 : 0;
    const int surplus = (on && off > 1) ? off - 1 : 0;
    int n_dead, n_src;
    const int dead_incl = block_scan_incl(dead, sc.redi, &n_dead, nw);
    const int sur_incl = block_scan_incl(surplus, sc.redi, (int*)nullptr, nw);
    const int src_incl = block_scan_incl(surplus > 0 ? 1 : 0, sc.redi, &n_src, nw);
    if (on) sc.Einc[i] = sur_incl;
    if (i == 0) {
        sc.base[0] = atomicAdd(a.n_moves, n_dead);
        sc.base[1] = atomicAdd(a.n_sources, n_src);
    }
    group_sync(nw);
    int mp = i;
    if (dead) {
        const int rank = dead_incl - 1;  // this dead slot takes surplus offspring number `rank`
        int lo = 0, hi = N;              // first j with Einc[j] > rank
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (sc.Einc[mid] > rank) hi = mid; else lo = mid + 1;
        }
        mp = lo < N ? lo : N - 1;
        a.dst_rows[sc.base[0] + rank] = r;
    }
    if (surplus > 0) {
        MoveSource ms;
        ms.src_row = r;
        ms.len = ln;
        ms.dst_begin = sc.base[0] + (sur_incl - surplus);
        ms.n_dst = surplus;
        a.sources[sc.base[1] + src_incl - 1] = ms;
    }

    // ---- copy particle state by the map, uniform weights ----
    if (on) {
        a.logW[r] = 0.0;
        a.S[r] = sc.S[mp];
        a.done_out[r] = sc.done[mp];
        a.len[r] = sc.len[mp];
        a.anc[r] = anc;
        a.map[r] = mp;
        a.hist_map[r] = mp;
        a.last_tok[r] = sc.tok[mp];
    }
    if (i == 0) a.logZ[g] += M + log(s1 / (double)N);
}

}  // namespace psmc
