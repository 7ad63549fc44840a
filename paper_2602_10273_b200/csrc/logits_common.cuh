// Shared pieces of the logit pass: the per-element arithmetic, the span triples the streaming
// kernel leaves behind, and the per-row finish (combine triples, draw the token, Eq. 7).
//
// For a row of logits l_0..l_{V-1} the pass needs
//   L1 = logsumexp(l)          normaliser of p = softmax(l)
//   Lb = logsumexp(beta l)     normaliser of the tempered proposal q of Corollary 1
//   y  = min{v : sum_{u<=v} exp(beta l_u) >= U sum_all}
//   log p(y) = l_y - L1,  log omega = alpha_t log p(y) - (beta l_y - Lb)     (Eq. 7 in logs)
// All exponentials are taken in base 2 (the hardware's ex2): with x_v = l_v * log2(e),
//   exp(l_v) = 2^{x_v}.  x_v - c is formed as fma(l, k_lo, fma(l, k_hi, -c)) with log2(e) = k_hi + k_lo split
// over two floats, so the product carries no representation error of log2(e) and the big parts cancel
// before the small one is added.  k_hi has 16 significant bits: l k_hi - c is then exact for the terms that matter
// (bf16 logits, c close to l k_hi), and l k_lo is far larger than the spacing of floats near x - c, so the one
// rounding that is left is unbiased.  (With k_hi = float(log2 e) the small part, 2e-8 l, was below half that
// spacing for most terms and simply dropped out of the sum: every x low by 2e-8 l, the dominant terms of a row low
// by about 3e-8 of their value, always in the same direction.)  The streaming kernel cuts a row into spans and writes one triple (c, s1, sb)
// per span:   c = a reference exponent (close to the span's largest x),  s1 = sum 2^{x - c},
//   sb = sum 2^{beta (x - c)}.  Reference exponents are whole numbers.
// The finish rescales the triples to the row's largest c in fp64, in span order, finds the span
// that holds U * sum_all by a prefix sum over the sb terms, and re-reads only that span.
#pragma once

#include <cuda_bf16.h>

#include "common.cuh"

namespace psmc {

constexpr float kNegBig = -3.3895313892515355e38f;  // most negative finite bf16; start value of a running maximum
constexpr float kRefFloor = -3.0e38f;               // reference exponent of a lane or span that saw no finite logit
constexpr float kLog2eHi = 1.44268798828125f;       // log2 e to 16 significant bits: its product with a bf16 logit is exact
constexpr float kLog2eLo = 7.052607543300837e-6f;   // float(log2 e - kLog2eHi); what is left is 1.7e-13
constexpr double kLn2 = 0.6931471805599453;

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

// x - c for one logit: l * log2(e) - c
__device__ __forceinline__ float rel_exponent(float l, float neg_c) {
    return fmaf(l, kLog2eLo, fmaf(l, kLog2eHi, neg_c));
}
// Reference exponent for logits bounded by m: m * log2(e) rounded up to a whole number (so that rescaling between
// reference points is an exact power of two) plus `shift`, kept finite.  shift = 1 (ref_shift) puts every exponent
// x - c at or below -1, where the hardware's 2^x has one known mean error (kEx2Low, below); between -1 and 0 and above
// 0 its mean error is a different one, and sums that mix the ranges cannot be corrected.
__device__ __forceinline__ float ref_exponent(float m, float shift) { return fmaxf(ceilf(m * kLog2eHi) + shift, kRefFloor); }
// The shift costs range at the bottom: the largest term of a sum may then be as small as 2^{-2 - slack log2 e}, its
// beta-th power 2^{-4.9 beta} with the slack of the streaming kernel.  Up to beta = 16 that stays far above the
// smallest normal float; beyond, the reference is left where it is and the sums are not corrected.
constexpr float kMaxShiftBeta = 16.f;
__host__ __device__ __forceinline__ float ref_shift(float bf) { return bf <= kMaxShiftBeta ? 1.f : 0.f; }

// ex2.approx.ftz.f32 returns 2^x low by this fraction of the value on average for x <= -1 (B200, 2^26 arguments per
// range against exp2 in fp64: -4.95e-8 ... -5.08e-8 for every range [-k-1, -k), k = 1 ... 59; -2.2e-8 on [-1, 0),
// +0.6e-8 on [0, 1), +3.3e-8 above).  A sum of such terms is low by the same fraction whatever the terms are, and a
// sum of their beta-th powers formed by squaring (exactly rounded multiplications) by beta times that.  Left in, the
// error is the same at every token and adds up in log p(y_{1:t}): 3.4e-8 per token, 1e-4 after 2900 tokens.
constexpr double kEx2Low = 4.99e-8;
// what to add to ln(sum 2^{x-c}) and ln(sum 2^{beta (x-c)}) as the kernels form them
template <int MODE>
__device__ __forceinline__ void ln_sum_corrections(double beta, double& add_s1, double& add_sb) {
    if (ref_shift((float)beta) == 0.f) {
        add_s1 = add_sb = 0.0;
        return;
    }
    add_s1 = kEx2Low;
    add_sb = (MODE == kBeta1 || MODE == kBetaAny) ? kEx2Low : beta * kEx2Low;  // one ex2 per term, or one squared up
}

// 2^{beta d} for d = x - c.  One MUFU: for beta in {1,2,4,8} 2^d is squared up; bf = (float)beta otherwise.
template <int MODE>
__device__ __forceinline__ float mass_beta(float d, float bf) {
    if (MODE == kBetaAny) return ex2(d * bf);
    float e = ex2(d);
    if (MODE == kBeta1) return e;
    e *= e;
    if (MODE == kBeta2) return e;
    e *= e;
    if (MODE == kBeta4) return e;
    return e * e;
}
// mass 2^{beta (x - C)} of one logit
template <int MODE>
__device__ __forceinline__ float logit_mass(float l, float neg_C, float bf) {
    return mass_beta<MODE>(rel_exponent(l, neg_C), bf);
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
    const float4* partials;  // [R][n_spans] = (c, s1, sb, -)
    double beta, alpha_t;
    float bf;                // (float)beta
    int vec;                 // rows are 16-byte aligned
};

struct RowResult {
    int tok;       // -1 when the row is unusable
    double logp;   // log p(y)
    double loginc; // log omega
};

// What one warp learns from a row's span triples.  Every lane holds the same values.
struct RowTotals {
    bool ok;        // false: NaN, +inf, or no finite logit
    float C;        // the row's largest reference exponent
    double S1, Sb;  // sum 2^{x - C}, sum 2^{beta (x - C)}
    double target;  // U * Sb
    double base;    // mass of the spans before span `jsel`
    int jsel;       // span that holds the target
};

// 2^e for a whole number e <= 0, exactly, built from its bits; 0 below the normal range (such a term is less than
// 2^-1022 of the row's largest and cannot change any sum)
__device__ __forceinline__ double pow2_neg(int e) { return e >= -1022 ? __hiloint2double((1023 + e) << 20, 0) : 0.0; }

// 2^{dc} and 2^{beta dc} for a span whose reference exponent lies dc <= 0 below the row's.  dc is a whole number,
// so for whole beta both factors are exact powers of two; other beta take one fp64 exp2.
template <int MODE>
__device__ __forceinline__ void span_scales(float dcf, double beta, double& f1, double& fb) {
    const int dc = (int)fmaxf(dcf, -4000.f);  // below -1022 every factor is 0
    f1 = pow2_neg(dc);
    if (MODE == kBeta1) fb = f1;
    else if (MODE == kBeta2) fb = pow2_neg(2 * dc);
    else if (MODE == kBeta4) fb = pow2_neg(4 * dc);
    else if (MODE == kBeta8) fb = pow2_neg(8 * dc);
    else fb = exp2(beta * (double)dc);
}

// When the row is one part of a longer row (a vocabulary shard): the reference exponent of the whole row, the
// target mass in that scale, and the mass of everything before this part.
struct RowFrame {
    float C;
    double target, base;
};

// Totals, target and selected span out of n triples handed out by fetch(j) (global memory, shared memory: the
// arithmetic and its order are the same wherever the numbers come from); one warp, every lane gets the same result.
// FRAMED: the triples are rescaled to fr->C instead of the row's own largest reference exponent, the prefix over the
// spans starts at fr->base and looks for fr->target (U is not used).
template <int MODE, bool FRAMED = false, class Fetch>
__device__ __forceinline__ RowTotals combine_triples(Fetch fetch, int n, double beta, double U, int lane,
                                                     const RowFrame* fr = nullptr) {
    constexpr int kKeep = 8;  // span masses a lane keeps in registers between the two sweeps (rows of <= 256 spans)
    RowTotals t;
    t.ok = false;

    // the lane's first triple is fetched once and kept (rows of up to 32 spans need no second trip to L2)
    const float4 f0 = lane < n ? fetch(lane) : make_float4(kRefFloor, 0.f, 0.f, 0.f);
    float cf = kRefFloor;
    if (FRAMED) {
        cf = fr->C;
    } else {
        cf = f0.x;
        for (int j = lane + 32; j < n; j += 32) cf = fmaxf(cf, fetch(j).x);
        cf = warp_max(cf);
    }
    t.C = cf;

    // totals, every term rescaled to the row's reference in fp64
    double a_sum = 0.0, b_sum = 0.0;
    double keep[kKeep];
#pragma unroll
    for (int i = 0; i < kKeep; ++i) keep[i] = 0.0;
    for (int j = lane, i = 0; j < n; j += 32, ++i) {
        const float4 f = i == 0 ? f0 : fetch(j);
        double f1, fb;
        span_scales<MODE>(f.x - cf, beta, f1, fb);
        const double a = (double)f.y * f1;
        const double b = (MODE == kBeta1) ? a : (double)f.z * fb;
        a_sum += a;
        b_sum += b;
#pragma unroll
        for (int q = 0; q < kKeep; ++q)
            if (q == i) keep[q] = b;
    }
    t.S1 = warp_sum(a_sum);
    t.Sb = warp_sum(b_sum);
    if (!FRAMED && (!(t.S1 > 0.0) || !(t.Sb > 0.0) || isinf(t.S1) || isinf(t.Sb))) return t;

    // span that holds the target: inclusive prefix over spans in order, 32 spans per round
    t.target = FRAMED ? fr->target : U * t.Sb;
    double carry = FRAMED ? fr->base : 0.0, base = 0.0, last_base = 0.0;
    int jsel = -1, last_pos = -1;
    for (int c = 0, i = 0; c < n && jsel < 0; c += 32, ++i) {
        const int j = c + lane;
        double b = 0.0;
        if (i < kKeep) {
#pragma unroll
            for (int q = 0; q < kKeep; ++q)
                if (q == i) b = keep[q];
        } else if (j < n) {
            const float4 f = fetch(j);
            double f1, fb;
            span_scales<MODE>(f.x - cf, beta, f1, fb);
            b = (MODE == kBeta1) ? (double)f.y * f1 : (double)f.z * fb;
        }
        const double incl = carry + warp_scan_incl(b, lane);
        const unsigned hit = __ballot_sync(kFull, b > 0.0 && incl >= t.target);
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
    if (jsel < 0) return t;
    t.jsel = jsel;
    t.base = base;
    t.ok = true;
    return t;
}

// The same for up to 32 triples, one per lane, in straight-line code: lane j passes triple j (lanes from n on pass
// any triple with zero sums).  The same additions in the same order as combine_triples.
template <int MODE>
__device__ __forceinline__ RowTotals combine_triples_32(float4 f, double beta, double U, int lane) {
    RowTotals t;
    t.ok = false;
    const float cf = warp_max(f.x);
    t.C = cf;
    double f1, fb;
    span_scales<MODE>(f.x - cf, beta, f1, fb);
    const double a = (double)f.y * f1;
    const double b = (MODE == kBeta1) ? a : (double)f.z * fb;
    t.S1 = warp_sum(a);
    t.Sb = warp_sum(b);
    if (!(t.S1 > 0.0) || !(t.Sb > 0.0) || isinf(t.S1) || isinf(t.Sb)) return t;
    t.target = U * t.Sb;
    const double incl = warp_scan_incl(b, lane);
    const unsigned hit = __ballot_sync(kFull, b > 0.0 && incl >= t.target);
    const unsigned pos = __ballot_sync(kFull, b > 0.0);
    if (!pos) return t;
    const int src = hit ? __ffs(hit) - 1 : 31 - __clz(pos);  // the last span with mass if rounding leaves every prefix short
    t.jsel = src;
    t.base = __shfl_sync(kFull, incl - b, src);
    t.ok = true;
    return t;
}

// the triples of row `row` as the streaming kernel left them in global memory
template <int MODE, bool FRAMED = false>
__device__ __forceinline__ RowTotals combine_spans(const FinishParams& p, int row, double U, int lane,
                                                   const RowFrame* fr = nullptr) {
    const float4* P = p.partials + (size_t)row * p.n_spans;
    return combine_triples<MODE, FRAMED>([&](int j) { return __ldcg(&P[j]); }, p.n_spans, p.beta, U, lane, fr);
}

// One lane's share of the selected span: `E` consecutive logits from e0 (clipped to b0).  Returns their mass
// (eight logits summed in fp32 at a time, then in fp64).
template <int DT, int MODE, int BATCH = 4>
__device__ __forceinline__ double lane_share(const FinishParams& p, const void* rowp, int e0, int E, int b0, float neg_C) {
    constexpr int kPer = DT == PSMC_BF16 ? 8 : 4;  // logits per 16 bytes
    double lm = 0.0;
    if (e0 >= b0) return lm;
    if (p.vec && e0 + E <= b0) {
        const uint4* q = reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(rowp) + (size_t)e0 * (16 / kPer));
        const int Q = E / kPer;
        for (int q0 = 0; q0 < Q; q0 += BATCH) {  // BATCH loads in flight
            uint4 v[BATCH];
#pragma unroll
            for (int i = 0; i < BATCH; ++i)
                if (q0 + i < Q) v[i] = q[q0 + i];
#pragma unroll
            for (int i = 0; i < BATCH; ++i) {
                if (q0 + i >= Q) break;
                const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
                float g[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (DT == PSMC_BF16)
                        g[j] = logit_mass<MODE>(__uint_as_float(w[j] << 16), neg_C, p.bf) +
                               logit_mass<MODE>(__uint_as_float(w[j] & 0xffff0000u), neg_C, p.bf);
                    else
                        g[j] = logit_mass<MODE>(__uint_as_float(w[j]), neg_C, p.bf);
                }
                lm += (double)((g[0] + g[1]) + (g[2] + g[3]));
            }
        }
    } else {
        const int e1 = min(b0, e0 + E);
        for (int i = e0; i < e1; ++i) lm += (double)logit_mass<MODE>(load_elem<DT>(rowp, i), neg_C, p.bf);
    }
    return lm;
}

// Last position of [a0, b0) whose logit has mass, -1 if none (one warp; the rare case in which the re-read sums fall
// a rounding error short of the target).
template <int DT, int MODE>
__device__ __forceinline__ int last_with_mass(const FinishParams& p, const void* rowp, int a0, int b0, float neg_C, int lane) {
    int last = -1;
    for (int i = a0 + lane; i < b0; i += 32)
        if (logit_mass<MODE>(load_elem<DT>(rowp, i), neg_C, p.bf) > 0.f) last = i;
    return warp_max(last);
}

// Token inside the owner lane's logits [o0, o1): 32 at a time across the warp, in vocabulary order, the loads of
// up to four rounds issued together.  `run` is the mass before o0.  Returns -1 only if nothing there has mass.
template <int DT, int MODE>
__device__ __forceinline__ int locate_in_lane(const FinishParams& p, const void* rowp, int o0, int o1, double run,
                                              double target, float neg_C, int lane) {
    int y = -1, last_with_mass = -1;
    for (int c0 = o0; c0 < o1 && y < 0; c0 += 128) {
        float l[4];
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int i = c0 + 32 * b + lane;
            l[b] = i < o1 ? load_elem<DT>(rowp, i) : -INFINITY;
        }
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            if (c0 + 32 * b >= o1 || y >= 0) break;
            const float e = logit_mass<MODE>(l[b], neg_C, p.bf);  // -inf gives mass 0
            const double incl = run + warp_scan_incl((double)e, lane);
            const unsigned h3 = __ballot_sync(kFull, e > 0.f && incl >= target);
            const unsigned p3 = __ballot_sync(kFull, e > 0.f);
            if (h3) y = c0 + 32 * b + __ffs(h3) - 1;
            else if (p3) last_with_mass = c0 + 32 * b + 31 - __clz(p3);
            run = __shfl_sync(kFull, incl, 31);
        }
    }
    return y >= 0 ? y : last_with_mass;  // the finer sums may fall a rounding error short of the lane's total
}

// Called by all 32 lanes; every lane returns the same RowResult.  The two logarithms are taken side by side
// (lane 0 and lane 1 of one call) rather than one after the other.
template <int DT, int MODE>
__device__ __forceinline__ RowResult row_result(const FinishParams& p, const void* rowp, const RowTotals& t, int y, int lane) {
    RowResult r;
    // l_y - C ln 2: the token's logit relative to the row's reference, in natural units
    const double dl = (double)load_elem<DT>(rowp, y) - (double)t.C * kLn2;
    const double lg = log((lane & 1) ? t.Sb : t.S1);
    double add_s1, add_sb;
    ln_sum_corrections<MODE>(p.beta, add_s1, add_sb);
    const double ln_s1 = __shfl_sync(kFull, lg, 0) + add_s1, ln_sb = __shfl_sync(kFull, lg, 1) + add_sb;
    r.tok = y;
    r.logp = dl - ln_s1;  // log p(y) = l_y - L1
    // alpha_t log p(y) - log q(y), log q(y) = beta l_y - Lb, grouped so that the token's own logit drops out
    // exactly when beta = alpha_t (Theorem 1)
    r.loginc = (p.alpha_t - p.beta) * dl - p.alpha_t * ln_s1 + ln_sb;
    return r;
}

// The token inside span t.jsel, by one warp: every lane sums its share of the span, the lane whose share reaches the
// target is searched 32 logits at a time.  Every lane returns the same position (-1: nothing in the span has mass).
template <int DT, int MODE>
__device__ __forceinline__ int locate_token_warp(const FinishParams& p, const void* rowp, const RowTotals& t, int lane) {
    const float neg_C = -t.C;
    const int a0 = t.jsel * p.span, b0 = min(p.V, a0 + p.span);
    const int E = p.span >> 5;
    const double lm = lane_share<DT, MODE>(p, rowp, a0 + lane * E, E, b0, neg_C);
    const double r_incl = t.base + warp_scan_incl(lm, lane);
    const unsigned hit2 = __ballot_sync(kFull, lm > 0.0 && r_incl >= t.target);
    if (hit2) {
        const int owner = __ffs(hit2) - 1;
        const double run = __shfl_sync(kFull, r_incl - lm, owner);
        const int o0 = a0 + owner * E;
        return locate_in_lane<DT, MODE>(p, rowp, o0, min(b0, o0 + E), run, t.target, neg_C, lane);
    }
    return last_with_mass<DT, MODE>(p, rowp, a0, b0, neg_C, lane);  // the re-read sums fall short of the target
}

// ---- the finish of one row by one warp on its own (no shared memory, no CTA barrier) ----
// Every lane returns the same RowResult.
template <int DT, int MODE>
__device__ __forceinline__ RowResult finish_row_warp(const FinishParams& p, int row, double U, int lane) {
    const RowResult bad{-1, 0.0, 0.0};
    const RowTotals t = combine_spans<MODE>(p, row, U, lane);
    if (!t.ok) return bad;
    const void* rowp = reinterpret_cast<const char*>(p.logits) + (size_t)row * p.ld * (DT == PSMC_F32 ? 4 : 2);
    const int y = locate_token_warp<DT, MODE>(p, rowp, t, lane);
    if (y < 0) return bad;
    return row_result<DT, MODE>(p, rowp, t, y, lane);
}

// ---- the finish at CTA level: several warps share a row ----
constexpr int kFinishMaxWarps = 32;
struct FinishShared {
    RowTotals row[kFinishMaxWarps];  // per row of the current pass: what its first warp learnt from the triples
    bool live[kFinishMaxWarps];      // does the row need finishing at all
    double tot[kFinishMaxWarps];     // mass of the part of the selected span each warp re-read
};

// warps per row: as many as the CTA can spare, each part of the span at least 256 logits (8 per lane)
__host__ __device__ inline int finish_warps_per_row(int n_rows, int span, int n_warps) {
    int w = 1;
    while (w * 2 * n_rows <= n_warps && w * 2 <= 8 && span / (w * 2) >= 256) w *= 2;
    return w;
}

// Every thread of the CTA calls this (it synchronises the CTA).  Finishes rows row0 .. row0+n_rows-1, n_warps/wpr
// rows at a time: one warp per row combines the span triples, then `wpr` warps (a power of two) share the re-read of
// the selected span, then the warp whose part holds the target pins the token down.  live(k): does row k need
// finishing; uniform(k): its U; emit(k, result) is called by lane 0 of one warp per finished row.
template <int DT, int MODE, class LiveFn, class UniformFn, class EmitFn>
__device__ __forceinline__ void finish_rows(const FinishParams& p, FinishShared& sh, int row0, int n_rows, int wpr,
                                            LiveFn live, UniformFn uniform, EmitFn emit) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const int rows_per_pass = n_warps / wpr;
    const int q = warp & (wpr - 1), kk = warp / wpr;  // this warp's part of the span, and its row within the pass
    for (int k0 = 0; k0 < n_rows; k0 += rows_per_pass) {
        // ---- one warp per row: totals, target, span ----
        if (warp < rows_per_pass) {
            const int k = k0 + warp;
            // the triples are fetched whether or not the row turns out to be live: the two loads overlap
            RowTotals t;
            t.ok = false;
            if (k < n_rows) t = combine_spans<MODE>(p, row0 + k, uniform(k), lane);
            const bool lv = k < n_rows && live(k);
            if (lane == 0) {
                sh.live[warp] = lv;
                sh.row[warp] = t;
            }
        }
        __syncthreads();
        // ---- wpr warps per row: mass of each part of the selected span ----
        const int k = k0 + kk;
        const bool active = kk < rows_per_pass && sh.live[kk];
        const void* rowp = reinterpret_cast<const char*>(p.logits) + (size_t)(row0 + k) * p.ld * (DT == PSMC_F32 ? 4 : 2);
        RowTotals t;
        t.ok = false;
        double lm = 0.0, incl = 0.0;
        int a0 = 0, b0 = 0, E = 0, sub = 0;
        float neg_C = 0.f;
        if (active) {
            t = sh.row[kk];
            if (t.ok) {
                neg_C = -t.C;
                a0 = t.jsel * p.span;
                b0 = min(p.V, a0 + p.span);
                sub = p.span / wpr;
                E = sub >> 5;
                lm = lane_share<DT, MODE>(p, rowp, a0 + q * sub + lane * E, E, b0, neg_C);
                incl = warp_scan_incl(lm, lane);
            }
            if (lane == 31) sh.tot[warp] = incl;
        }
        __syncthreads();
        // ---- the warp whose part reaches the target: the token ----
        if (active) {
            const int w0 = warp - q;  // first warp of this row
            if (!t.ok) {
                if (q == 0 && lane == 0) emit(k, RowResult{-1, 0.0, 0.0});
            } else {
                // which part of the span reaches the target: same additions, in the same order, in every warp
                double cum = t.base, before = t.base;
                int first_hit = -1;
                for (int i = 0; i < wpr; ++i) {
                    if (i == q) before = cum;
                    const double ti = sh.tot[w0 + i];
                    cum += ti;
                    if (first_hit < 0 && ti > 0.0 && cum >= t.target) first_hit = i;
                }
                int y = -1;
                bool mine = false;
                if (first_hit == q) {
                    mine = true;
                    const double r_incl = before + incl;
                    const unsigned hit2 = __ballot_sync(kFull, lm > 0.0 && r_incl >= t.target);
                    const int owner = hit2 ? __ffs(hit2) - 1 : 31;
                    const double run = __shfl_sync(kFull, r_incl - lm, owner);
                    const int o0 = a0 + q * sub + owner * E;
                    y = locate_in_lane<DT, MODE>(p, rowp, o0, min(b0, o0 + E), run, t.target, neg_C, lane);
                } else if (first_hit < 0 && q == 0) {
                    mine = true;  // the re-read sums fall short of the target: last token with mass in the span
                    y = last_with_mass<DT, MODE>(p, rowp, a0, b0, neg_C, lane);
                }
                if (mine) {
                    RowResult rr{-1, 0.0, 0.0};
                    if (y >= 0) rr = row_result<DT, MODE>(p, rowp, t, y, lane);
                    if (lane == 0) emit(k, rr);
                }
            }
        }
        __syncthreads();  // sh is reused by the next pass; the emitted results are visible to the CTA
    }
}

}  // namespace psmc
