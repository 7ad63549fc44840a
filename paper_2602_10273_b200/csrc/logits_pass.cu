// Logit pass of the Power-SMC step: per live row, in ONE sweep over the V logits,
//   L1 = logsumexp(l)            (log-softmax normaliser of p, Eq. 7 numerator)
//   Lb = logsumexp(beta * l)     (normaliser of the tempered proposal q of Corollary 1)
//   y  = min{v : sum_{u<=v} exp(beta l_u) >= U * sum_all}   (inverse CDF in vocabulary order)
//   log p(y), log omega = alpha_t log p(y) - log q(y)        (Eq. 7 in logs)
//
// Work decomposition.  A row is cut into spans of `span` consecutive logits; one warp streams one
// span with 128-bit loads (8 bf16 / 4 fp32 per lane per load, four loads in flight per lane) and keeps,
// per lane, a running maximum m and the sums  s1 = sum exp(l - m),  sb = sum exp(beta (l - m)).
// One MUFU.EX2 per element: for beta in {1,2,4,8} exp(beta d) is exp(d) squared up; other beta
// (exponent-bridging steps) pay a second EX2.  A warp writes one (m, s1, sb) triple per span and
// takes a ticket on the row's counter; the warp that takes the last ticket finishes the row:
// it rescales the span triples to the row maximum in fp64 in span order (so the result does not
// depend on which warp arrived when), prefix-sums the sb terms to find the span that holds
// U * sum_all, and re-reads only that span (a few KB, normally an L2 hit) to find the token.
// HBM traffic is therefore one read of the logits.  No spin-waits anywhere: the ticket is wait-free.
#include <cuda_bf16.h>

#include "common.cuh"
#include "internal.h"

namespace psmc {
namespace {

constexpr float kNegBig = -3.3895313892515355e38f;  // most negative finite bf16; stands in for -inf as a start value
constexpr float kLog2e = 1.4426950408889634f;
constexpr int kThreads = 256;
constexpr int kWarpsPerCta = kThreads / 32;
constexpr int kCtasPerSm = 4;

enum BetaMode { kBeta1 = 0, kBeta2 = 1, kBeta4 = 2, kBeta8 = 3, kBetaAny = 4 };

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// exp(beta * d) for d = l - m <= 0, in the arithmetic of the chosen mode
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
// one element into the two running sums
template <int MODE>
__device__ __forceinline__ void accumulate(float d, float cb, float& s1, float& sb) {
    float e = ex2(d * kLog2e);
    s1 += e;
    if (MODE == kBeta2) {
        sb = fmaf(e, e, sb);
    } else if (MODE == kBeta4) {
        float e2 = e * e;
        sb = fmaf(e2, e2, sb);
    } else if (MODE == kBeta8) {
        float e2 = e * e;
        float e4 = e2 * e2;
        sb = fmaf(e4, e4, sb);
    } else if (MODE == kBetaAny) {
        sb += ex2(d * cb);
    }
}
template <int MODE>
__device__ __forceinline__ void raise_max(float cm, float cb, float& m, float& s1, float& sb) {
    if (cm > m) {
        float d0 = m - cm;  // <= 0; -inf-ish on the first call, which zeroes the (empty) sums
        s1 *= ex2(d0 * kLog2e);
        if (MODE != kBeta1) sb *= mass_beta<MODE>(d0, cb);
        m = cm;
    }
}

template <int DT>
__device__ __forceinline__ float load_elem(const void* base, int64_t i) {
    if (DT == PSMC_F32) return __ldg(reinterpret_cast<const float*>(base) + i);
    uint32_t b = __ldg(reinterpret_cast<const unsigned short*>(base) + i);
    return __uint_as_float(b << 16);
}

struct LaneSums {
    float m, s1, sb;
};

// ---- bf16, 16-byte aligned span: 8 logits per lane per load ----
template <int MODE, int NW>
__device__ __forceinline__ void consume_bf16(const uint32_t (&w)[NW], float cb, LaneSums& a, __nv_bfloat162& m2) {
    __nv_bfloat162 pm = *reinterpret_cast<const __nv_bfloat162*>(&w[0]);
#pragma unroll
    for (int i = 1; i < NW; ++i) pm = __hmax2(pm, *reinterpret_cast<const __nv_bfloat162*>(&w[i]));
    if (!__hble2(pm, m2)) {  // some logit exceeds the running maximum (rare after the first loads)
        float cm = fmaxf(__low2float(pm), __high2float(pm));
        raise_max<MODE>(cm, cb, a.m, a.s1, a.sb);
        m2 = __float2bfloat162_rn(a.m);  // exact: m is itself a bf16 value
    }
#pragma unroll
    for (int i = 0; i < NW; ++i) {
        float lo = __uint_as_float(w[i] << 16);
        float hi = __uint_as_float(w[i] & 0xffff0000u);
        accumulate<MODE>(lo - a.m, cb, a.s1, a.sb);
        accumulate<MODE>(hi - a.m, cb, a.s1, a.sb);
    }
}
template <int MODE>
__device__ __forceinline__ void span_bf16_vec(const unsigned short* row, int a0, int b0, float cb, int lane,
                                              LaneSums& acc) {
    const int n = b0 - a0, n_chunks = n >> 3;
    const uint4* p = reinterpret_cast<const uint4*>(row + a0);
    __nv_bfloat162 m2 = __float2bfloat162_rn(acc.m);
    int c = lane;
    for (; c + 96 < n_chunks; c += 128) {
        uint4 v0 = ld_stream16(p + c), v1 = ld_stream16(p + c + 32), v2 = ld_stream16(p + c + 64),
              v3 = ld_stream16(p + c + 96);
        uint32_t w[16] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w,
                          v2.x, v2.y, v2.z, v2.w, v3.x, v3.y, v3.z, v3.w};
        consume_bf16<MODE, 16>(w, cb, acc, m2);
    }
    for (; c < n_chunks; c += 32) {
        uint4 v0 = ld_stream16(p + c);
        uint32_t w[4] = {v0.x, v0.y, v0.z, v0.w};
        consume_bf16<MODE, 4>(w, cb, acc, m2);
    }
    const int tail = n & 7;  // ragged end of the row
    if (lane < tail) {
        float x = load_elem<PSMC_BF16>(row, (int64_t)a0 + (n_chunks << 3) + lane);
        raise_max<MODE>(x, cb, acc.m, acc.s1, acc.sb);
        accumulate<MODE>(x - acc.m, cb, acc.s1, acc.sb);
    }
}

// ---- fp32, 16-byte aligned span: 4 logits per lane per load ----
template <int MODE, int NX>
__device__ __forceinline__ void consume_f32(const float (&x)[NX], float cb, LaneSums& a) {
    float cm = x[0];
#pragma unroll
    for (int i = 1; i < NX; ++i) cm = fmaxf(cm, x[i]);
    raise_max<MODE>(cm, cb, a.m, a.s1, a.sb);
#pragma unroll
    for (int i = 0; i < NX; ++i) accumulate<MODE>(x[i] - a.m, cb, a.s1, a.sb);
}
template <int MODE>
__device__ __forceinline__ void span_f32_vec(const float* row, int a0, int b0, float cb, int lane, LaneSums& acc) {
    const int n = b0 - a0, n_chunks = n >> 2;
    const uint4* p = reinterpret_cast<const uint4*>(row + a0);
    int c = lane;
    for (; c + 96 < n_chunks; c += 128) {
        uint4 v0 = ld_stream16(p + c), v1 = ld_stream16(p + c + 32), v2 = ld_stream16(p + c + 64),
              v3 = ld_stream16(p + c + 96);
        float x[16] = {__uint_as_float(v0.x), __uint_as_float(v0.y), __uint_as_float(v0.z), __uint_as_float(v0.w),
                       __uint_as_float(v1.x), __uint_as_float(v1.y), __uint_as_float(v1.z), __uint_as_float(v1.w),
                       __uint_as_float(v2.x), __uint_as_float(v2.y), __uint_as_float(v2.z), __uint_as_float(v2.w),
                       __uint_as_float(v3.x), __uint_as_float(v3.y), __uint_as_float(v3.z), __uint_as_float(v3.w)};
        consume_f32<MODE, 16>(x, cb, acc);
    }
    for (; c < n_chunks; c += 32) {
        uint4 v0 = ld_stream16(p + c);
        float x[4] = {__uint_as_float(v0.x), __uint_as_float(v0.y), __uint_as_float(v0.z), __uint_as_float(v0.w)};
        consume_f32<MODE, 4>(x, cb, acc);
    }
    const int tail = n & 3;
    if (lane < tail) {
        float x = load_elem<PSMC_F32>(row, (int64_t)a0 + (n_chunks << 2) + lane);
        raise_max<MODE>(x, cb, acc.m, acc.s1, acc.sb);
        accumulate<MODE>(x - acc.m, cb, acc.s1, acc.sb);
    }
}

// ---- any alignment: one logit per lane per load ----
template <int DT, int MODE>
__device__ __forceinline__ void span_scalar(const void* row, int a0, int b0, float cb, int lane, LaneSums& acc) {
    for (int i = a0 + lane; i < b0; i += 32) {
        float x = load_elem<DT>(row, i);
        raise_max<MODE>(x, cb, acc.m, acc.s1, acc.sb);
        accumulate<MODE>(x - acc.m, cb, acc.s1, acc.sb);
    }
}

struct Params {
    const void* logits;
    int R, V;
    int64_t ld;
    int span, n_spans;
    float cb;  // beta * log2(e)
    double beta, alpha_t;
    const double* u;
    uint64_t seed;
    int t, N;
    const uint8_t* done;
    unsigned int* counters;  // [R]
    float4* partials;        // [R][n_spans] = (m, s1, sb, -)
    int32_t* tok;
    double* logp;
    double* loginc;
    int32_t* status;
    int32_t* zero_words;
};

// The warp that took a row's last ticket: combine the span triples, draw the token, write the row's results.
template <int DT, int MODE>
__device__ void finish_row(const Params& p, int row, int lane) {
    const int n = p.n_spans;
    const float4* P = p.partials + (size_t)row * n;
    const void* rowp = reinterpret_cast<const char*>(p.logits) + (size_t)row * p.ld * (DT == PSMC_F32 ? 4 : 2);

    float mf = kNegBig;
    for (int j = lane; j < n; j += 32) mf = fmaxf(mf, __ldcg(&P[j]).x);
    mf = warp_max(mf);
    const double M = (double)mf;

    // lane owns the contiguous block of spans [j0, j1): sums in span order, fp64
    const int per = (n + 31) >> 5;
    const int j0 = min(n, lane * per), j1 = min(n, j0 + per);
    double a_sum = 0.0, b_sum = 0.0;
    for (int j = j0; j < j1; ++j) {
        float4 f = __ldcg(&P[j]);
        double dm = (double)f.x - M;
        a_sum += (double)f.y * exp(dm);
        b_sum += (double)(MODE == kBeta1 ? f.y : f.z) * exp(p.beta * dm);
    }
    const double S1 = warp_sum(a_sum);
    const double b_incl = warp_scan_incl(b_sum, lane);
    const double Sb = __shfl_sync(kFull, b_incl, 31);

    if (!(S1 > 0.0) || !(Sb > 0.0) || isinf(S1) || isinf(Sb)) {  // NaN, +inf, or nothing finite in the row
        if (lane == 0) {
            raise_status(p.status, PSMC_E_NUMERIC);
            p.tok[row] = -1;
            p.logp[row] = 0.0;
            p.loginc[row] = 0.0;
        }
        return;
    }

    double U;
    if (p.u) {
        U = p.u[row];
    } else {
        U = hash_uniform(hash5(p.seed, kStreamToken, (uint64_t)(row / p.N), (uint64_t)p.t, (uint64_t)(row % p.N)));
    }
    const double target = U * Sb;

    // which span holds the target: first lane whose inclusive prefix reaches it, then the span inside that lane
    unsigned hit = __ballot_sync(kFull, b_incl >= target && b_sum > 0.0);
    int owner = hit ? __ffs(hit) - 1 : -1;
    if (owner < 0) {  // rounding left every prefix short: take the last lane that holds mass
        unsigned any = __ballot_sync(kFull, b_sum > 0.0);
        owner = 31 - __clz(any);
    }
    int jsel = -1;
    double base = 0.0;
    if (lane == owner) {
        double run = b_incl - b_sum;
        int last_pos = -1;
        double last_base = run;
        for (int j = j0; j < j1; ++j) {
            float4 f = __ldcg(&P[j]);
            double term = (double)(MODE == kBeta1 ? f.y : f.z) * exp(p.beta * ((double)f.x - M));
            if (term > 0.0) {
                last_pos = j;
                last_base = run;
            }
            if (run + term >= target && term > 0.0) {
                jsel = j;
                base = run;
                break;
            }
            run += term;
        }
        if (jsel < 0) {
            jsel = last_pos;
            base = last_base;
        }
    }
    jsel = __shfl_sync(kFull, jsel, owner);
    base = __shfl_sync(kFull, base, owner);

    // re-read that span in vocabulary order: lane owns a contiguous run of `sub` logits
    const int a0 = jsel * p.span, b0 = min(p.V, a0 + p.span);
    const int sub = (b0 - a0 + 31) >> 5;
    const int e0 = min(b0, a0 + lane * sub), e1 = min(b0, e0 + sub);
    double lane_mass = 0.0;
    int lane_last_pos = -1;
    for (int i = e0; i < e1; ++i) {
        float e = mass_beta<MODE>(load_elem<DT>(rowp, i) - mf, p.cb);
        lane_mass += (double)e;
        if (e > 0.f) lane_last_pos = i;
    }
    const double r_incl = warp_scan_incl(lane_mass, lane);
    unsigned hit2 = __ballot_sync(kFull, base + r_incl >= target && lane_mass > 0.0);
    int y = -1;
    if (hit2) {
        const int owner2 = __ffs(hit2) - 1;
        if (lane == owner2) {
            double run = base + (r_incl - lane_mass);
            for (int i = e0; i < e1; ++i) {
                float e = mass_beta<MODE>(load_elem<DT>(rowp, i) - mf, p.cb);
                run += (double)e;
                if (e > 0.f) y = i;  // remembers the last token with mass in case rounding falls short
                if (run >= target && e > 0.f) break;
            }
        }
        y = __shfl_sync(kFull, y, owner2);
    } else {  // the re-read sums fall a rounding error short of the target: last token with mass in the span
        y = warp_max(lane_last_pos);
    }
    if (lane == 0) {
        if (y < 0) {
            raise_status(p.status, PSMC_E_NUMERIC);
            p.tok[row] = -1;
            p.logp[row] = 0.0;
            p.loginc[row] = 0.0;
        } else {
            const double dl = (double)load_elem<DT>(rowp, y) - M;
            const double ln_s1 = log(S1), ln_sb = log(Sb);
            p.tok[row] = y;
            p.logp[row] = dl - ln_s1;  // log p(y) = l_y - L1
            // alpha_t log p(y) - log q(y) with log q(y) = beta l_y - Lb, grouped so that the token's own
            // logit drops out exactly when beta = alpha_t (Theorem 1)
            p.loginc[row] = (p.alpha_t - p.beta) * dl - p.alpha_t * ln_s1 + ln_sb;
        }
    }
}

template <int DT, int MODE, bool VEC>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) logits_pass_kernel(const Params p) {
    const int lane = threadIdx.x & 31;
    const int warp_global = blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
    const int n_warps = gridDim.x * kWarpsPerCta;
    if (p.zero_words && blockIdx.x == 0 && threadIdx.x < 2) p.zero_words[threadIdx.x] = 0;

    const int64_t n_tasks = (int64_t)p.R * p.n_spans;
    for (int64_t task = warp_global; task < n_tasks; task += n_warps) {
        const int row = (int)(task / p.n_spans), sp = (int)(task - (int64_t)row * p.n_spans);
        if (p.done && p.done[row]) continue;  // absorbing state: the row's logits are never read
        const int a0 = sp * p.span, b0 = min(p.V, a0 + p.span);
        const void* rowp = reinterpret_cast<const char*>(p.logits) + (size_t)row * p.ld * (DT == PSMC_F32 ? 4 : 2);

        LaneSums acc{kNegBig, 0.f, 0.f};
        if (VEC) {
            if (DT == PSMC_BF16)
                span_bf16_vec<MODE>(reinterpret_cast<const unsigned short*>(rowp), a0, b0, p.cb, lane, acc);
            else
                span_f32_vec<MODE>(reinterpret_cast<const float*>(rowp), a0, b0, p.cb, lane, acc);
        } else {
            span_scalar<DT, MODE>(rowp, a0, b0, p.cb, lane, acc);
        }

        // one triple per span: rescale every lane to the warp's maximum, then add
        const float wm = warp_max(acc.m);
        const float d0 = acc.m - wm;
        float s1 = acc.s1 * ex2(d0 * kLog2e);
        float sb = (MODE == kBeta1) ? 0.f : acc.sb * mass_beta<MODE>(d0, p.cb);
        s1 = warp_sum(s1);
        sb = warp_sum(sb);

        unsigned int ticket = 0;
        if (lane == 0) {
            __stcg(&p.partials[(size_t)row * p.n_spans + sp], make_float4(wm, s1, sb, 0.f));
            __threadfence();
            ticket = atomicAdd(&p.counters[row], 1u);
        }
        ticket = __shfl_sync(kFull, ticket, 0);
        if (ticket == (unsigned)(p.n_spans - 1)) {
            __threadfence();
            if (lane == 0) p.counters[row] = 0;  // leave the scratch as it was found
            finish_row<DT, MODE>(p, row, lane);
        }
    }
}

typedef void (*KernelFn)(const Params);
template <int DT, bool VEC>
KernelFn pick_mode(int mode) {
    switch (mode) {
        case kBeta1: return logits_pass_kernel<DT, kBeta1, VEC>;
        case kBeta2: return logits_pass_kernel<DT, kBeta2, VEC>;
        case kBeta4: return logits_pass_kernel<DT, kBeta4, VEC>;
        case kBeta8: return logits_pass_kernel<DT, kBeta8, VEC>;
        default: return logits_pass_kernel<DT, kBetaAny, VEC>;
    }
}

size_t counters_bytes(int R) { return (((size_t)R * 4) + 255) / 256 * 256; }

}  // namespace

int logits_pass_span(int R, int V) {
    // about four tasks per resident warp when the problem is large enough, between 512 and 4096 logits each
    const int64_t resident_warps = (int64_t)kSMs * kCtasPerSm * kWarpsPerCta;
    int64_t want = ((int64_t)R * V) / (resident_warps * 4);
    int span = 512;
    while (span < 4096 && span * 2 <= want) span *= 2;
    return span;
}

size_t logits_pass_scratch_bytes(int R, int V) {
    const int span = logits_pass_span(R, V);
    const size_t n_spans = ((size_t)V + span - 1) / span;
    return counters_bytes(R) + (size_t)R * n_spans * sizeof(float4);
}

cudaError_t launch_logits_pass(const LogitsPassArgs& a, cudaStream_t stream) {
    Params p;
    p.logits = a.logits;
    p.R = a.R;
    p.V = a.V;
    p.ld = a.ld;
    p.span = logits_pass_span(a.R, a.V);
    p.n_spans = (a.V + p.span - 1) / p.span;
    p.beta = a.beta;
    p.alpha_t = a.alpha_t;
    p.cb = (float)(a.beta * 1.4426950408889634);
    p.u = a.u;
    p.seed = a.seed;
    p.t = a.t;
    p.N = a.N > 0 ? a.N : 1;
    p.done = a.done;
    p.counters = reinterpret_cast<unsigned int*>(a.scratch);
    p.partials = reinterpret_cast<float4*>(reinterpret_cast<char*>(a.scratch) + counters_bytes(a.R));
    p.tok = a.tok;
    p.logp = a.logp;
    p.loginc = a.loginc;
    p.status = a.status;
    p.zero_words = a.zero_words;

    int mode = kBetaAny;
    if (a.beta == 1.0) mode = kBeta1;
    else if (a.beta == 2.0) mode = kBeta2;
    else if (a.beta == 4.0) mode = kBeta4;
    else if (a.beta == 8.0) mode = kBeta8;

    const size_t esize = a.dt == PSMC_F32 ? 4 : 2;
    const bool vec = (reinterpret_cast<uintptr_t>(a.logits) % 16 == 0) && ((a.ld * esize) % 16 == 0) &&
                     ((p.span * esize) % 16 == 0);
    KernelFn fn;
    if (a.dt == PSMC_F32)
        fn = vec ? pick_mode<PSMC_F32, true>(mode) : pick_mode<PSMC_F32, false>(mode);
    else
        fn = vec ? pick_mode<PSMC_BF16, true>(mode) : pick_mode<PSMC_BF16, false>(mode);

    const int64_t n_tasks = (int64_t)a.R * p.n_spans;
    int64_t blocks = (n_tasks + kWarpsPerCta - 1) / kWarpsPerCta;
    const int64_t max_blocks = (int64_t)kSMs * kCtasPerSm;
    if (blocks > max_blocks) blocks = max_blocks;
    if (blocks < 1) blocks = 1;
    fn<<<(unsigned)blocks, kThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace psmc

extern "C" size_t psmc_logits_pass_scratch_bytes(int R, int V) {
    if (R < 1 || V < 2) return 0;
    return psmc::logits_pass_scratch_bytes(R, V);
}

extern "C" psmc_status psmc_logits_pass(const void* logits, psmc_dtype dt, int R, int V, int64_t ld, double beta,
                                        double alpha_t, const double* u, const uint8_t* done, void* scratch,
                                        size_t scratch_bytes, int32_t* tok, double* logp, double* loginc,
                                        int32_t* status_word, void* stream) {
    if (!logits || !u || !scratch || !tok || !logp || !loginc || !status_word) return PSMC_E_INVAL;
    if (R < 1 || V < 2 || ld < V || !(beta > 0.0) || !(alpha_t >= 1.0)) return PSMC_E_INVAL;
    if (dt != PSMC_F32 && dt != PSMC_BF16) return PSMC_E_INVAL;
    if (scratch_bytes < psmc::logits_pass_scratch_bytes(R, V) || reinterpret_cast<uintptr_t>(scratch) % 256 != 0)
        return PSMC_E_INVAL;
    psmc::LogitsPassArgs a{};
    a.logits = logits; a.dt = dt; a.R = R; a.V = V; a.ld = ld; a.beta = beta; a.alpha_t = alpha_t;
    a.u = u; a.seed = 0; a.t = 0; a.N = 1; a.done = done; a.scratch = scratch;
    a.tok = tok; a.logp = logp; a.loginc = loginc; a.status = status_word; a.zero_words = nullptr;
    return psmc::launch_logits_pass(a, static_cast<cudaStream_t>(stream)) == cudaSuccess ? PSMC_OK : PSMC_E_CUDA;
}
