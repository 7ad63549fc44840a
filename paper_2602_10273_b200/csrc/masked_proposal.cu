// The logit pass with the proposal restricted to a set S of tokens: the top_k tokens of the row by logit, or the
// nucleus holding a share top_p of the tempered distribution softmax(beta l).  Tokens rank by logit, lower id first
// among equal logits; S is the first k of that ranking.  Eq. 7 takes the proposal actually sampled from,
//   q_S(v) = exp(beta l_v) / sum_{u in S} exp(beta l_u) on S,   log omega = alpha_t log p(y) - log q_S(y),
// with p the softmax over the WHOLE row.
//
// One CTA per row.  A logit's bit pattern maps to an unsigned key that orders like the value, so S is
// {key > T} plus the first `need` tokens with key == T in id order.  (T, need) come from a radix search over the
// key, 8 bits a level from the top (2 levels for bf16, 4 for fp32): a level counts, per digit, the tokens whose
// higher digits equal the prefix found so far -- and for the nucleus their mass 2^{beta (x - C)} as a 64-bit
// fixed-point number (2^-40 units, integer adds: the totals do not depend on the order of the atomics) -- then picks
// the digit in which the running count reaches k (the running mass reaches top_p of the total).  Counters live in
// shared memory as [digit][lane] columns, so the lanes of a warp never meet on an address however the logits
// cluster.  Tokens with equal key have equal mass, so on the last level need = ceil(remaining mass / mass of one).
// Then two ordered sweeps (every warp owns a contiguous stretch of the row): the mass of S per warp, and, in the
// warp whose stretch holds U * sum, the token.  The row is read from HBM once; the other sweeps hit L2.
#include "internal.h"
#include "logits_common.cuh"
#include "weights_core.cuh"

namespace psmc {
namespace {

constexpr int kDigits = 256;
constexpr float kFixOne = 1099511627776.f;  // 2^40: fixed-point unit of the nucleus masses (masses are <= 1)
constexpr size_t kHistBytes = (size_t)kDigits * 32 * (sizeof(uint32_t) + sizeof(unsigned long long));

struct MaskedParams {
    const void* logits;
    int V;
    int64_t ld;
    int N, t;
    int top_k;      // > 0: top-k; 0: nucleus of share top_p
    double top_p;
    double beta, alpha_t;
    float bf;
    uint64_t seed;
    const uint8_t* done;
    int32_t* tok;
    double* logp;
    double* loginc;
    int32_t* set_size;    // [R] |S| of each live row
    int32_t* zero_words;  // two words cleared before anything else (may be NULL)
    int32_t* status;
};

template <int DT>
__device__ __forceinline__ uint32_t key_of(uint32_t b) {
    constexpr uint32_t sign = DT == PSMC_BF16 ? 0x8000u : 0x80000000u;
    constexpr uint32_t all = DT == PSMC_BF16 ? 0xffffu : 0xffffffffu;
    if (b == sign) b = 0;  // -0 ranks with +0
    return (b & sign) ? (~b & all) : (b | sign);
}
template <int DT>
__device__ __forceinline__ float value_of(uint32_t b) {
    return __uint_as_float(DT == PSMC_BF16 ? b << 16 : b);
}
template <int DT>
__device__ __forceinline__ uint32_t load_bits(const void* rowp, int i) {
    if (DT == PSMC_F32) return __ldg(reinterpret_cast<const uint32_t*>(rowp) + i);
    return __ldg(reinterpret_cast<const unsigned short*>(rowp) + i);
}

// f(bits) for every logit of the row, in no particular order: 16-byte loads between the first and the last
// 16-byte boundary, single loads for the ragged ends.
template <int DT, class F>
__device__ __forceinline__ void for_each_logit(const void* rowp, int V, F f) {
    constexpr int kPer = DT == PSMC_BF16 ? 8 : 4, kEs = DT == PSMC_BF16 ? 2 : 4;
    int head = (int)(((16 - (reinterpret_cast<uintptr_t>(rowp) & 15)) & 15) / kEs);
    if (head > V) head = V;
    const int nvec = (V - head) / kPer, tail0 = head + nvec * kPer;
    const uint4* q = reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(rowp) + (size_t)head * kEs);
    for (int j = threadIdx.x; j < nvec; j += blockDim.x) {
        const uint4 v = __ldg(&q[j]);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            if (DT == PSMC_BF16) {
                f(w[c] & 0xffffu);
                f(w[c] >> 16);
            } else {
                f(w[c]);
            }
        }
    }
    for (int i = threadIdx.x; i < head; i += blockDim.x) f(load_bits<DT>(rowp, i));
    for (int i = tail0 + threadIdx.x; i < V; i += blockDim.x) f(load_bits<DT>(rowp, i));
}

struct Selection {      // what the radix search has settled so far (shared, written by warp 0)
    uint32_t prefix;    // the digits chosen so far
    uint32_t k_rem;     // top-k: tokens still to take among those that match the prefix
    unsigned long long m_rem;  // nucleus: mass still to cover among those that match the prefix
    uint32_t above;     // tokens with a larger key than every token that matches the prefix
    uint32_t n_ties, need;     // after the last level
};

// Warp 0: pick the digit (from 255 down) in which the running count reaches k_rem / the running mass reaches m_rem.
__device__ __forceinline__ void pick_digit(Selection& sel, const uint32_t* tot_cnt, const unsigned long long* tot_mass,
                                           bool nucleus, bool first, bool last, double top_p, int lane) {
    uint32_t c_loc = 0;
    unsigned long long m_loc = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int d = 255 - (8 * lane + j);
        c_loc += tot_cnt[d];
        m_loc += tot_mass[d];
    }
    uint32_t c_run = warp_scan_incl(c_loc, lane) - c_loc;  // lane 0 holds the largest digits
    unsigned long long m_run = warp_scan_incl(m_loc, lane) - m_loc;
    uint32_t k_rem = sel.k_rem;
    unsigned long long m_rem = sel.m_rem;
    if (nucleus && first) {  // the share is taken of the whole row's mass, known once the first level is counted
        const unsigned long long total = __shfl_sync(kFull, m_run + m_loc, 31);
        m_rem = (unsigned long long)ceil(top_p * (double)total);
        if (m_rem < 1) m_rem = 1;
    }
    int dsel = -1, dlow = -1;
    uint32_t c_above = 0;
    unsigned long long m_above = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int d = 255 - (8 * lane + j);
        const uint32_t c = tot_cnt[d];
        const unsigned long long m = tot_mass[d];
        const bool here = nucleus ? (m > 0 && m_run + m >= m_rem) : (c > 0 && c_run + c >= k_rem);
        if (dsel < 0 && here) {
            dsel = d;
            c_above = c_run;
            m_above = m_run;
        }
        if (c > 0 && (!nucleus || m > 0)) dlow = d;  // lowest digit of this lane that could be chosen at all
        c_run += c;
        m_run += m;
    }
    const unsigned found = __ballot_sync(kFull, dsel >= 0);
    int src;
    if (found) {
        src = __ffs(found) - 1;
    } else {  // rounding left the running mass short of the target: everything counts, down to the last digit in use
        const unsigned any = __ballot_sync(kFull, dlow >= 0);
        src = any ? 31 - __clz(any) : 0;
        if (lane == src) {
            dsel = dlow >= 0 ? dlow : 0;
            c_above = 0;
            m_above = 0;
            for (int d = 255; d > dsel; --d) {
                c_above += tot_cnt[d];
                m_above += tot_mass[d];
            }
        }
    }
    dsel = __shfl_sync(kFull, dsel, src);
    c_above = __shfl_sync(kFull, c_above, src);
    m_above = __shfl_sync(kFull, m_above, src);
    if (lane == 0) {
        sel.prefix = (sel.prefix << 8) | (uint32_t)dsel;
        sel.above += c_above;
        sel.k_rem = k_rem > c_above ? k_rem - c_above : 1;
        sel.m_rem = m_rem > m_above ? m_rem - m_above : 1;
        if (last) {
            const uint32_t n = tot_cnt[dsel];
            uint32_t need;
            if (nucleus) {
                const unsigned long long one = n ? tot_mass[dsel] / n : 0;  // equal keys, equal masses
                need = one ? (uint32_t)min((unsigned long long)n, (sel.m_rem + one - 1) / one) : n;
            } else {
                need = sel.k_rem;
            }
            sel.n_ties = n;
            sel.need = need < 1 ? 1 : (need > n ? n : need);
        }
    }
}

template <int DT, int MODE>
__global__ void __launch_bounds__(1024, 1) masked_rows_kernel(const __grid_constant__ MaskedParams p) {
    extern __shared__ __align__(16) unsigned char hist_raw[];
    uint32_t* cnt = reinterpret_cast<uint32_t*>(hist_raw);                                       // [256][32]
    unsigned long long* mass = reinterpret_cast<unsigned long long*>(hist_raw + kDigits * 32 * 4);  // [256][32]
    __shared__ double red[33];
    __shared__ float redf[33];
    __shared__ uint32_t tot_cnt[kDigits];
    __shared__ unsigned long long tot_mass[kDigits];
    __shared__ Selection sel;
    __shared__ double wmass[32];
    __shared__ int wties[32];

    constexpr int kKeyBits = DT == PSMC_BF16 ? 16 : 32, kLevels = kKeyBits / 8;
    const int row = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const int V = p.V;
    chain_begin();
    if (p.zero_words && blockIdx.x == 0 && threadIdx.x < 2) p.zero_words[threadIdx.x] = 0;
    if (p.done[row]) return;
    const void* rowp = reinterpret_cast<const char*>(p.logits) + (size_t)row * p.ld * (DT == PSMC_F32 ? 4 : 2);
    const bool nucleus = p.top_k == 0;

    // ---- the row's largest logit; NaN and +inf make the row unusable ----
    float mx = -INFINITY;
    int bad = 0;
    for_each_logit<DT>(rowp, V, [&](uint32_t b) {
        const float l = value_of<DT>(b);
        bad |= (l != l) || l == INFINITY;
        mx = fmaxf(mx, l);
    });
    mx = block_max(mx, redf, nw);
    bad = __syncthreads_or(bad);
    if (bad || mx == -INFINITY) {
        if (threadIdx.x == 0) {
            raise_status(p.status, PSMC_E_NUMERIC);
            p.tok[row] = -1;
            p.logp[row] = 0.0;
            p.loginc[row] = 0.0;
            p.set_size[row] = 0;
        }
        return;
    }
    const float C = ref_exponent(mx), neg_C = -C;

    // ---- radix search for (T, need); the first level also sums 2^{x - C} over the whole row ----
    if (threadIdx.x == 0) {
        sel.prefix = 0;
        sel.k_rem = (uint32_t)min(p.top_k, V);
        sel.m_rem = 0;
        sel.above = 0;
    }
    double s1 = 0.0;
    uint32_t prefix = 0;
    for (int level = 0; level < kLevels; ++level) {
        const int shift = kKeyBits - 8 * (level + 1);
        for (int i = threadIdx.x; i < kDigits * 32; i += blockDim.x) {
            cnt[i] = 0;
            if (nucleus) mass[i] = 0;
        }
        __syncthreads();
        for_each_logit<DT>(rowp, V, [&](uint32_t b) {
            const float l = value_of<DT>(b);
            if (level == 0) s1 += (double)ex2(rel_exponent(l, neg_C));
            const uint32_t key = key_of<DT>(b);
            if (level > 0 && (key >> (shift + 8)) != prefix) return;
            const uint32_t d = (key >> shift) & 255u;
            atomicAdd(&cnt[d * 32 + lane], 1u);
            if (nucleus)
                atomicAdd(&mass[d * 32 + lane], __float2ull_rn(logit_mass<MODE>(l, neg_C, p.bf) * kFixOne));
        });
        __syncthreads();
        for (int d = threadIdx.x; d < kDigits; d += blockDim.x) {
            uint32_t c = 0;
            unsigned long long m = 0;
            for (int j = 0; j < 32; ++j) {
                c += cnt[d * 32 + j];
                if (nucleus) m += mass[d * 32 + j];
            }
            tot_cnt[d] = c;
            tot_mass[d] = m;
        }
        __syncthreads();
        if (warp == 0) pick_digit(sel, tot_cnt, tot_mass, nucleus, level == 0, level == kLevels - 1, p.top_p, lane);
        __syncthreads();
        prefix = sel.prefix;
    }
    const double S1 = block_sum(s1, red, nw);
    const uint32_t T = prefix, need = sel.need;
    const bool all_ties = need == sel.n_ties;
    const int set_size = (int)(sel.above + need);

    // ---- ordered sweeps: warp w owns logits [lo, hi) ----
    const int seg = (((V + nw - 1) / nw) + 31) & ~31;
    const int lo = min(V, warp * seg), hi = min(V, lo + seg);
    int tie_base = 0;
    if (!all_ties) {  // ties at T are taken in id order: how many lie before this warp's stretch
        int n = 0;
        for (int base = lo; base < hi; base += 32) {
            const int i = base + lane;
            const bool tie = i < hi && key_of<DT>(load_bits<DT>(rowp, i)) == T;
            n += __popc(__ballot_sync(kFull, tie));
        }
        if (lane == 0) wties[warp] = n;
        __syncthreads();
        for (int w = 0; w < warp; ++w) tie_base += wties[w];
    }
    // is token i (key, tie rank within the row) in S
    auto in_set = [&](uint32_t key, bool tie, int rank) { return key > T || (tie && (all_ties || (uint32_t)rank < need)); };
    {
        double acc = 0.0;
        int tb = tie_base;
        for (int base = lo; base < hi; base += 32) {
            const int i = base + lane;
            const bool valid = i < hi;
            const uint32_t b = valid ? load_bits<DT>(rowp, i) : 0u;
            const uint32_t key = key_of<DT>(b);
            const bool tie = valid && key == T;
            const unsigned bal = __ballot_sync(kFull, tie);
            const int rank = tb + __popc(bal & ((1u << lane) - 1u));
            tb += __popc(bal);
            if (valid && in_set(key, tie, rank)) acc += (double)logit_mass<MODE>(value_of<DT>(b), neg_C, p.bf);
        }
        acc = warp_sum(acc);
        if (lane == 0) wmass[warp] = acc;
    }
    __syncthreads();
    double Sb = 0.0;
    for (int w = 0; w < nw; ++w) Sb += wmass[w];
    const int g = row / p.N, k = row - g * p.N;
    const double U = hash_uniform(hash5(p.seed, kStreamToken, (uint64_t)g, (uint64_t)p.t, (uint64_t)k));
    const double target = U * Sb;
    int wsel = -1, wlast = -1;
    double run0 = 0.0, run_last = 0.0;
    {
        double cum = 0.0;
        for (int w = 0; w < nw; ++w) {
            const double m = wmass[w];
            if (m > 0.0) {
                if (wsel < 0 && cum + m >= target) {
                    wsel = w;
                    run0 = cum;
                }
                wlast = w;
                run_last = cum;
            }
            cum += m;
        }
        if (wsel < 0) {
            wsel = wlast;
            run0 = run_last;
        }
    }
    if (warp != wsel) return;  // (wsel >= 0: the row's largest logit is in S and has mass)

    // ---- the warp that holds the target: the token ----
    int y = -1, last_pos = -1;
    double run = run0;
    int tb = tie_base;
    for (int base = lo; base < hi && y < 0; base += 32) {
        const int i = base + lane;
        const bool valid = i < hi;
        const uint32_t b = valid ? load_bits<DT>(rowp, i) : 0u;
        const uint32_t key = key_of<DT>(b);
        const bool tie = valid && key == T;
        const unsigned bal = __ballot_sync(kFull, tie);
        const int rank = tb + __popc(bal & ((1u << lane) - 1u));
        tb += __popc(bal);
        const double e = (valid && in_set(key, tie, rank)) ? (double)logit_mass<MODE>(value_of<DT>(b), neg_C, p.bf) : 0.0;
        const double incl = run + warp_scan_incl(e, lane);
        const unsigned hit = __ballot_sync(kFull, e > 0.0 && incl >= target);
        const unsigned pos = __ballot_sync(kFull, e > 0.0);
        if (hit) y = base + __ffs(hit) - 1;
        else if (pos) last_pos = base + 31 - __clz(pos);
        run = __shfl_sync(kFull, incl, 31);
    }
    if (y < 0) y = last_pos;  // the finer sums fell a rounding error short of the warp's total
    if (lane == 0) {
        if (y < 0) {
            raise_status(p.status, PSMC_E_NUMERIC);
            p.tok[row] = -1;
            p.logp[row] = 0.0;
            p.loginc[row] = 0.0;
        } else {
            const double dl = (double)load_elem<DT>(rowp, y) - (double)C * kLn2;
            const double ln_s1 = log(S1), ln_sb = log(Sb);
            p.tok[row] = y;
            p.logp[row] = dl - ln_s1;
            p.loginc[row] = (p.alpha_t - p.beta) * dl - p.alpha_t * ln_s1 + ln_sb;
        }
        p.set_size[row] = set_size;
    }
}

// ---- the per-group update from row results that are already in memory ----
__global__ void __launch_bounds__(1024) rows_weights_kernel(const __grid_constant__ WeightsArgs a) {
    __shared__ GroupScratch<kMaxParticles> sc;
    const int g = blockIdx.x, i = threadIdx.x, N = a.N;
    chain_begin();
    ParticleState st{};
    int tk = -1;
    double lp = 0.0, inc = 0.0;
    if (i < N) {
        const int r = g * N + i;
        st = load_particle(a, r);
        if (!st.done) {
            tk = a.tok[r];
            lp = a.logp[r];
            inc = a.loginc[r];
        }
    }
    group_update(a, g, i, (N + 31) >> 5, sc, tk, lp, inc, st);
}

typedef void (*MaskedFn)(const MaskedParams);
template <int DT>
MaskedFn pick_masked(int mode) {
    switch (mode) {
        case kBeta1: return masked_rows_kernel<DT, kBeta1>;
        case kBeta2: return masked_rows_kernel<DT, kBeta2>;
        case kBeta4: return masked_rows_kernel<DT, kBeta4>;
        case kBeta8: return masked_rows_kernel<DT, kBeta8>;
        default: return masked_rows_kernel<DT, kBetaAny>;
    }
}

}  // namespace

cudaError_t launch_step_masked(const LogitsStreamArgs& la, const WeightsArgs& wa, int top_k, double top_p,
                               int32_t* set_size, cudaStream_t stream) {
    MaskedParams p;
    p.logits = la.logits; p.V = la.V; p.ld = la.ld; p.N = wa.N; p.t = wa.t; p.top_k = top_k; p.top_p = top_p;
    p.beta = wa.beta; p.alpha_t = wa.alpha_t; p.bf = (float)wa.beta; p.seed = wa.seed; p.done = la.done;
    p.tok = wa.tok; p.logp = wa.logp; p.loginc = wa.loginc; p.set_size = set_size; p.zero_words = la.zero_words;
    p.status = la.status;
    const int mode = beta_mode(wa.beta);
    MaskedFn fn = la.dt == PSMC_F32 ? pick_masked<PSMC_F32>(mode) : pick_masked<PSMC_BF16>(mode);
    cudaError_t e = allow_dynamic_smem(reinterpret_cast<const void*>(fn), (int)kHistBytes);
    if (e != cudaSuccess) return e;
    const int threads = la.V >= 16384 ? 1024 : 256;
    e = launch_chained(fn, dim3((unsigned)la.R), dim3((unsigned)threads), kHistBytes, stream, p);
    if (e != cudaSuccess) return e;
    const int warps = (wa.N + 31) >> 5;
    return launch_chained(rows_weights_kernel, dim3((unsigned)wa.G), dim3((unsigned)(warps * 32)), 0, stream, wa);
}

}  // namespace psmc
