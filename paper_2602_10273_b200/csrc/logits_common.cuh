// Shared pieces of the logit pass: the per-element arithmetic, the span triples the streaming
// kernel leaves behind, and the per-row finish (combine triples, draw the token, Eq. 7).
//
// For a row of logits l_0..l_{V-1} the pass needs
//   L1 = logsumexp(l)          normaliser of p = softmax(l)
//   Lb = logsumexp(beta l)     normaliser of the tempered proposal q of Corollary 1
//   y  = min{v : sum_{u<=v} exp(beta l_u) >= U sum_all}
//   log p(y) = l_y - L1,  log omega = alpha_t log p(y) - (beta l_y - Lb)     (Eq. 7 in logs)
// The streaming kernel cuts a row into spans and writes one triple (m, s1, sb) per span:
//   m = max l over the span, s1 = sum exp(l - m), sb = sum exp(beta (l - m)).
// finish_row() rescales the triples to the row maximum in fp64, in span order, finds the span
// that holds U * sum_all by a prefix sum over the sb terms, and re-reads only that span.
#pragma once

#include <cuda_bf16.h>

#include "common.cuh"

namespace psmc {

constexpr float kNegBig = -3.3895313892515355e38f;  // most negative finite bf16; start value of a running maximum
constexpr float kLog2e = 1.4426950408889634f;

enum BetaMode { kBeta1 = 0, kBeta2 = 1, kBeta4 = 2, kBeta8 = 3, kBetaAny = 4 };

__host__ inline int beta_mode(double beta) {
    if (beta == 1.0) return kBeta1;
    if (beta == 2.0) return kBeta2;
    if (beta == 4.0) return kBeta4;
    if (beta == 8.0) return kBeta8;
    return kBetaAny;
}

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// exp(beta * d) for d = l - m <= 0.  One MUFU: for beta in {1,2,4,8} exp(d) is squared up.
template <int MODE>
__device__ __forceinline__ float mass_beta(float d, float cb) {
    if (MODE == kBetaAny) return ex2(d * cb);
    float e = ex2(d * kLog2e);
    if (MODE == kBeta1) return e;
    e *= e;
    if (MODE == kBeta2) return e;
    e *= e;
    if (MODE == kBeta4) return e;
    return e * e;
}

template <int DT>
__device__ __forceinline__ float load_elem(const void* base, int64_t i) {
    if (DT == PSMC_F32) return __ldg(reinterpret_cast<const float*>(base) + i);
    uint32_t b = __ldg(reinterpret_cast<const unsigned short*>(base) + i);
    return __uint_as_float(b << 16);
}

struct FinishParams {
    const void* logits;
    int V;
    int64_t ld;
    int span, n_spans;
    const float4* partials;  // [R][n_spans] = (m, s1, sb, -)
    double beta, alpha_t;
    float cb;                // beta * log2(e)
    int vec;                 // rows are 16-byte aligned
};

struct RowResult {
    int tok;       // -1 when the row is unusable
    double logp;   // log p(y)
    double loginc; // log omega
};

// One warp finishes one row.  Every lane returns the same RowResult.
template <int DT, int MODE>
__device__ __forceinline__ RowResult finish_row(const FinishParams& p, int row, double U, int lane) {
    RowResult bad{-1, 0.0, 0.0};
    const int n = p.n_spans;
    const float4* P = p.partials + (size_t)row * n;
    const void* rowp = reinterpret_cast<const char*>(p.logits) + (size_t)row * p.ld * (DT == PSMC_F32 ? 4 : 2);

    // row maximum
    float mf = kNegBig;
    for (int j = lane; j < n; j += 32) mf = fmaxf(mf, __ldcg(&P[j]).x);
    mf = warp_max(mf);
    const double M = (double)mf;

    // totals, every term rescaled to the row maximum in fp64
    double a_sum = 0.0, b_sum = 0.0;
    for (int j = lane; j < n; j += 32) {
        const float4 f = __ldcg(&P[j]);
        const double dm = (double)f.x - M;
        const double a = (double)f.y * exp(dm);
        a_sum += a;
        b_sum += (MODE == kBeta1) ? a : (double)f.z * exp(p.beta * dm);
    }
    const double S1 = warp_sum(a_sum), Sb = warp_sum(b_sum);
    if (!(S1 > 0.0) || !(Sb > 0.0) || isinf(S1) || isinf(Sb)) return bad;  // NaN, +inf, or nothing finite

    // span that holds the target: inclusive prefix over spans in order, 32 spans per round
    const double target = U * Sb;
    double carry = 0.0, base = 0.0, last_base = 0.0;
    int jsel = -1, last_pos = -1;
    for (int c = 0; c < n && jsel < 0; c += 32) {
        const int j = c + lane;
        double b = 0.0;
        if (j < n) {
            const float4 f = __ldcg(&P[j]);
            const double dm = (double)f.x - M;
            b = (MODE == kBeta1) ? (double)f.y * exp(dm) : (double)f.z * exp(p.beta * dm);
        }
        const double incl = carry + warp_scan_incl(b, lane);
        const unsigned hit = __ballot_sync(kFull, b > 0.0 && incl >= target);
        const unsigned pos = __ballot_sync(kFull, b > 0.0);
        if (hit) {
            const int src = __ffs(hit) - 1;
            jsel = c + src;
            base = __shfl_sync(kFull, incl - b, src);
        } else if (pos) {  // remember the last span with mass in case rounding leaves every prefix short
            const int src = 31 - __clz(pos);
            last_pos = c + src;
            last_base = __shfl_sync(kFull, incl - b, src);
        }
        carry = __shfl_sync(kFull, incl, 31);
    }
    if (jsel < 0) {
        jsel = last_pos;
        base = last_base;
    }
    if (jsel < 0) return bad;

    // re-read that span in vocabulary order: lane owns `sub` consecutive logits
    const int a0 = jsel * p.span, b0 = min(p.V, a0 + p.span);
    const int sub = p.span >> 5;
    const int e0 = a0 + lane * sub;
    float lane_mass = 0.f;
    int lane_last = -1;
    if (DT == PSMC_BF16 && p.vec && e0 + sub <= b0) {
        const uint4* q = reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned short*>(rowp) + e0);
        for (int k = 0; k < (sub >> 3); k += 2) {  // sub is a multiple of 16 (span >= 512)
            const uint4 v0 = q[k], v1 = q[k + 1];
            const uint32_t w[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
            float g = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float m0 = mass_beta<MODE>(__uint_as_float(w[i] << 16) - mf, p.cb);
                const float m1 = mass_beta<MODE>(__uint_as_float(w[i] & 0xffff0000u) - mf, p.cb);
                if (m0 > 0.f) lane_last = e0 + (k << 3) + 2 * i;
                if (m1 > 0.f) lane_last = e0 + (k << 3) + 2 * i + 1;
                g += m0 + m1;
            }
            lane_mass += g;
        }
    } else {
        const int e1 = min(b0, e0 + sub);
        for (int i = e0; i < e1; ++i) {
            const float e = mass_beta<MODE>(load_elem<DT>(rowp, i) - mf, p.cb);
            if (e > 0.f) lane_last = i;
            lane_mass += e;
        }
    }
    const double lm = (double)lane_mass;
    const double r_incl = base + warp_scan_incl(lm, lane);
    const unsigned hit2 = __ballot_sync(kFull, lm > 0.0 && r_incl >= target);
    int y = -1;
    if (hit2) {
        // the owner's `sub` logits, 32 at a time across the warp, in order
        const int owner = __ffs(hit2) - 1;
        double run = __shfl_sync(kFull, r_incl - lm, owner);
        const int o0 = a0 + owner * sub, o1 = min(b0, o0 + sub);
        int last_in_owner = -1;
        for (int c = o0; c < o1 && y < 0; c += 32) {
            const int i = c + lane;
            const float e = i < o1 ? mass_beta<MODE>(load_elem<DT>(rowp, i) - mf, p.cb) : 0.f;
            const double incl = run + warp_scan_incl((double)e, lane);
            const unsigned h3 = __ballot_sync(kFull, e > 0.f && incl >= target);
            const unsigned p3 = __ballot_sync(kFull, e > 0.f);
            if (h3) y = c + __ffs(h3) - 1;
            else if (p3) last_in_owner = c + 31 - __clz(p3);
            run = __shfl_sync(kFull, incl, 31);
        }
        if (y < 0) y = last_in_owner;  // the finer sums fell a rounding error short
    } else {
        y = warp_max(lane_last);       // the re-read sums fall short of the target: last token with mass
    }
    if (y < 0) return bad;

    RowResult r;
    const double dl = (double)load_elem<DT>(rowp, y) - M;
    const double ln_s1 = log(S1), ln_sb = log(Sb);
    r.tok = y;
    r.logp = dl - ln_s1;  // log p(y) = l_y - L1
    // alpha_t log p(y) - log q(y), log q(y) = beta l_y - Lb, grouped so that the token's own logit drops out
    // exactly when beta = alpha_t (Theorem 1)
    r.loginc = (p.alpha_t - p.beta) * dl - p.alpha_t * ln_s1 + ln_sb;
    return r;
}

// run-time dispatch of finish_row over the beta mode (the dtype stays a template parameter of the caller)
template <int DT>
__device__ __forceinline__ RowResult finish_row_mode(int mode, const FinishParams& p, int row, double U, int lane) {
    switch (mode) {
        case kBeta1: return finish_row<DT, kBeta1>(p, row, U, lane);
        case kBeta2: return finish_row<DT, kBeta2>(p, row, U, lane);
        case kBeta4: return finish_row<DT, kBeta4>(p, row, U, lane);
        case kBeta8: return finish_row<DT, kBeta8>(p, row, U, lane);
        default: return finish_row<DT, kBetaAny>(p, row, U, lane);
    }
}

}  // namespace psmc
