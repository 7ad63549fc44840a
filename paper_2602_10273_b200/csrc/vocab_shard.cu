// The step with the vocabulary split over P ranks (a tensor-parallel LM head leaves rank p with columns
// [v0_p, v0_p + V_p) of every logit row).  Particle state is replicated: every rank runs the per-group update on
// the same numbers and reaches the same bits, so only the logit pass needs an exchange, and a small one.
//
//   sweep    the streaming kernel over the local columns (logits_stream.cuh), then one triple per row
//            (C_p, S1_p, Sb_p) = (largest reference exponent, sum 2^{x - C_p}, sum 2^{beta (x - C_p)}) in fp64
//   -- all-gather of the triples: 24 bytes per row per rank --
//   locate   every rank forms the row totals from the P triples in rank order, hence the same target U * Sb and the
//            same owner (the first rank whose inclusive mass prefix reaches the target, the last rank with mass if
//            rounding leaves every prefix short); the owner walks its own spans from that prefix on, re-reads one
//            span and names the token; it publishes (token id in the whole vocabulary, the token's logit)
//   -- all-gather of the picks: 8 bytes per row per rank --
//   finish   log p(y) and log omega (Eq. 7) from the totals and the owner's pick, then the per-group update of
//            weights_core.cuh, identically on every rank
// The inverse CDF runs over the vocabulary in its natural order (rank 0's columns first), so the drawn token is the
// one the unsharded step draws up to the rounding of the partial sums.
#include "internal.h"
#include "logits_common.cuh"
#include "weights_core.cuh"

namespace psmc {
namespace {

constexpr int kRowsPerCta = 8;  // one warp per row

// Row totals out of the P triples, by one thread, in rank order: every rank, and both kernels below, take the same
// additions in the same order.
struct ShardTotals {
    bool ok;
    float C;
    double S1, Sb, target, base;
    int owner;
};
// get(p, C, s1, sb) hands out rank p's triple of the row (from registers, shared memory or global memory: the
// arithmetic and its order are the same wherever the numbers are fetched from).
template <int MODE, class Get>
__device__ __forceinline__ ShardTotals shard_combine(Get get, int P, double beta, double U) {
    ShardTotals t;
    t.ok = false;
    t.owner = -1;
    t.base = 0.0;
    double C = (double)kRefFloor;
    for (int p = 0; p < P; ++p) {
        double c, s1, sb;
        get(p, c, s1, sb);
        C = fmax(C, c);
    }
    t.C = (float)C;
    double S1 = 0.0, Sb = 0.0;
    for (int p = 0; p < P; ++p) {
        double c, s1, sb, f1, fb;
        get(p, c, s1, sb);
        span_scales<MODE>((float)(c - C), beta, f1, fb);
        S1 += s1 * f1;
        Sb += sb * fb;
    }
    t.S1 = S1;
    t.Sb = Sb;
    if (!(S1 > 0.0) || !(Sb > 0.0) || isinf(S1) || isinf(Sb)) return t;
    t.target = U * Sb;
    double incl = 0.0, last_base = 0.0;
    int last = -1;
    for (int p = 0; p < P; ++p) {
        double c, s1, sb, f1, fb;
        get(p, c, s1, sb);
        span_scales<MODE>((float)(c - C), beta, f1, fb);
        const double b = sb * fb;
        if (b > 0.0) {
            if (t.owner < 0 && incl + b >= t.target) {
                t.owner = p;
                t.base = incl;
            }
            last = p;
            last_base = incl;
        }
        incl += b;
    }
    if (t.owner < 0) {
        t.owner = last;
        t.base = last_base;
    }
    t.ok = t.owner >= 0;
    return t;
}
// rank p's triple of `row` straight from the gathered array
struct TriplesInGlobal {
    const double* all;
    int R, row;
    __device__ __forceinline__ void operator()(int p, double& c, double& s1, double& sb) const {
        const double* tr = all + ((size_t)p * R + row) * 3;
        c = __ldcg(&tr[0]);
        s1 = __ldcg(&tr[1]);
        sb = __ldcg(&tr[2]);
    }
};

// ---- sweep, second half: the span triples of the local columns become one triple per row ----
template <int MODE>
__global__ void __launch_bounds__(kRowsPerCta * 32) shard_triples_kernel(const float4* partials, int n_spans, double beta,
                                                                         int R, const uint8_t* done, double* out) {
    chain_begin();
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * kRowsPerCta + (threadIdx.x >> 5);
    if (row >= R) return;
    double C = (double)kRefFloor, s1 = 0.0, sb = 0.0;
    if (!done[row]) {
        const float4* P = partials + (size_t)row * n_spans;
        float cf = kRefFloor;
        for (int j = lane; j < n_spans; j += 32) cf = fmaxf(cf, __ldcg(&P[j]).x);
        cf = warp_max(cf);
        double a_sum = 0.0, b_sum = 0.0;
        for (int j = lane; j < n_spans; j += 32) {
            const float4 f = __ldcg(&P[j]);
            double f1, fb;
            span_scales<MODE>(f.x - cf, beta, f1, fb);
            const double a = (double)f.y * f1;
            a_sum += a;
            b_sum += (MODE == kBeta1) ? a : (double)f.z * fb;
        }
        s1 = warp_sum(a_sum);
        sb = warp_sum(b_sum);
        C = (double)cf;
    }
    if (lane == 0) {
        out[(size_t)row * 3 + 0] = C;
        out[(size_t)row * 3 + 1] = s1;
        out[(size_t)row * 3 + 2] = sb;
    }
}

// ---- locate: the owner of each row names the token ----
struct LocateParams {
    FinishParams f;  // the local columns
    const double* all;
    int P, rank, R, N, t, v0;
    int tile_width;  // > 0: every row is located in the columns given for it, which start at owner * tile_width
    uint64_t seed;
    const uint8_t* done;
    psmc_shard_pick* picks;
};
template <int DT, int MODE>
__global__ void __launch_bounds__(kRowsPerCta * 32) shard_locate_kernel(const __grid_constant__ LocateParams lp) {
    chain_begin();
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * kRowsPerCta + (threadIdx.x >> 5);
    if (row >= lp.R) return;
    psmc_shard_pick pick{-1, 0.f};
    if (!lp.done[row]) {
        const int g = row / lp.N, k = row - g * lp.N;
        const double U = hash_uniform(hash5(lp.seed, kStreamToken, (uint64_t)g, (uint64_t)lp.t, (uint64_t)k));
        ShardTotals st;
        if (lp.P <= 32) {  // lane p fetches rank p's triple: one round trip instead of one per rank
            double c = (double)kRefFloor, s1 = 0.0, sb = 0.0;
            if (lane < lp.P) TriplesInGlobal{lp.all, lp.R, row}(lane, c, s1, sb);
            st = shard_combine<MODE>(
                [&](int p, double& c_, double& s1_, double& sb_) {
                    c_ = __shfl_sync(kFull, c, p);
                    s1_ = __shfl_sync(kFull, s1, p);
                    sb_ = __shfl_sync(kFull, sb, p);
                },
                lp.P, lp.f.beta, U);
        } else {
            st = shard_combine<MODE>(TriplesInGlobal{lp.all, lp.R, row}, lp.P, lp.f.beta, U);
        }
        if (st.ok && (lp.tile_width > 0 || st.owner == lp.rank)) {
            const RowFrame fr{st.C, st.target, st.base};
            const RowTotals t = combine_spans<MODE, true>(lp.f, row, U, lane, &fr);
            if (t.ok) {
                const void* rowp =
                    reinterpret_cast<const char*>(lp.f.logits) + (size_t)row * lp.f.ld * (DT == PSMC_F32 ? 4 : 2);
                const int y = locate_token_warp<DT, MODE>(lp.f, rowp, t, lane);
                if (y >= 0) {
                    pick.tok = (lp.tile_width > 0 ? st.owner * lp.tile_width : lp.v0) + y;
                    pick.logit = load_elem<DT>(rowp, y);
                }
            }
        }
    }
    if (lane == 0) lp.picks[row] = pick;
}

// ---- finish: Eq. 7 from the totals and the owner's pick, then the group update ----
struct ShardFinishParams {
    WeightsArgs a;
    const double* all;
    const psmc_shard_pick* picks;  // [P][R]
    int P;
    int staged;  // the group's triples fit the dynamic shared memory given to the launch
    int picks_per_row;  // picks is [R]: row r's pick, whoever owns the row
};
template <int MODE>
__global__ void __launch_bounds__(1024) shard_weights_kernel(const __grid_constant__ ShardFinishParams sp) {
    __shared__ GroupScratch<kMaxParticles> sc;
    extern __shared__ double staged[];  // [N][P][3] when sp.staged: the group's triples, fetched by the whole CTA at once
    const WeightsArgs& a = sp.a;
    const int g = blockIdx.x, i = threadIdx.x, N = a.N;
    chain_begin();
    if (sp.staged) {
        const int per_rank = N * 3;
        for (int j = threadIdx.x; j < sp.P * per_rank; j += blockDim.x) {
            const int p = j / per_rank, rem = j - p * per_rank, k = rem / 3, q = rem - 3 * k;
            staged[(k * sp.P + p) * 3 + q] = __ldcg(&sp.all[((size_t)p * a.R + (size_t)g * N + k) * 3 + q]);
        }
        __syncthreads();
    }
    const bool on = i < N;
    ParticleState st{};
    int tk = -1;
    double lp = 0.0, inc = 0.0;
    if (on) {
        const int r = g * N + i;
        st = load_particle(a, r);
        if (!st.done) {
            const double U = hash_uniform(hash5(a.seed, kStreamToken, (uint64_t)g, (uint64_t)a.t, (uint64_t)i));
            ShardTotals tot;
            if (sp.staged) {
                const double* mine = staged + (size_t)i * sp.P * 3;
                tot = shard_combine<MODE>(
                    [&](int p, double& c, double& s1, double& sb) {
                        c = mine[3 * p];
                        s1 = mine[3 * p + 1];
                        sb = mine[3 * p + 2];
                    },
                    sp.P, a.beta, U);
            } else {
                tot = shard_combine<MODE>(TriplesInGlobal{sp.all, a.R, r}, sp.P, a.beta, U);
            }
            if (tot.ok) {
                const psmc_shard_pick pk = sp.picks[sp.picks_per_row ? (size_t)r : (size_t)tot.owner * a.R + r];
                if (pk.tok >= 0) {
                    // same grouping as the unsharded finish: the token's own logit drops out when beta = alpha_t
                    const double dl = (double)pk.logit - (double)tot.C * kLn2;
                    double add_s1, add_sb;
                    ln_sum_corrections<MODE>(a.beta, add_s1, add_sb);
                    const double ln_s1 = log(tot.S1) + add_s1, ln_sb = log(tot.Sb) + add_sb;
                    tk = pk.tok;
                    lp = dl - ln_s1;
                    inc = (a.alpha_t - a.beta) * dl - a.alpha_t * ln_s1 + ln_sb;
                }
            }
            if (tk < 0) raise_status(a.status, PSMC_E_NUMERIC);
        }
    }
    group_update(a, g, i, (N + 31) >> 5, sc, tk, lp, inc, st);
}

// ---- which part holds each row's target: what a caller that feeds the parts one after the other has to bring back ----
template <int MODE>
__global__ void __launch_bounds__(256) shard_owner_columns_kernel(const double* all, int P, int R, int N, int t, double beta,
                                                                  uint64_t seed, const uint8_t* done, int tile_width,
                                                                  int32_t* need_out) {
    chain_begin();
    const int row = blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= R) return;
    int need = -1;
    if (!done[row]) {
        const int g = row / N, k = row - g * N;
        const double U = hash_uniform(hash5(seed, kStreamToken, (uint64_t)g, (uint64_t)t, (uint64_t)k));
        const ShardTotals st = shard_combine<MODE>(TriplesInGlobal{all, R, row}, P, beta, U);
        if (st.ok) need = st.owner * tile_width;
    }
    need_out[row] = need;
}

template <int DT>
void (*pick_locate(int mode))(const LocateParams) {
    switch (mode) {
        case kBeta1: return shard_locate_kernel<DT, kBeta1>;
        case kBeta2: return shard_locate_kernel<DT, kBeta2>;
        case kBeta4: return shard_locate_kernel<DT, kBeta4>;
        case kBeta8: return shard_locate_kernel<DT, kBeta8>;
        default: return shard_locate_kernel<DT, kBetaAny>;
    }
}

}  // namespace

cudaError_t launch_shard_triples(const LogitsStreamArgs& la, double* triples_out, cudaStream_t stream) {
    const LogitsGeometry g = logits_geometry(la.logits, la.dt, la.R, la.V, la.ld, la.beta);
    void (*fn)(const float4*, int, double, int, const uint8_t*, double*);
    switch (g.mode) {
        case kBeta1: fn = shard_triples_kernel<kBeta1>; break;
        case kBeta2: fn = shard_triples_kernel<kBeta2>; break;
        case kBeta4: fn = shard_triples_kernel<kBeta4>; break;
        case kBeta8: fn = shard_triples_kernel<kBeta8>; break;
        default: fn = shard_triples_kernel<kBetaAny>; break;
    }
    return launch_chained(fn, dim3((unsigned)((la.R + kRowsPerCta - 1) / kRowsPerCta)), dim3(kRowsPerCta * 32), 0, stream,
                          reinterpret_cast<const float4*>(la.scratch), g.n_spans, la.beta, la.R, la.done, triples_out);
}

cudaError_t launch_shard_locate(const LogitsStreamArgs& la, const ShardLocateArgs& sa, cudaStream_t stream) {
    const LogitsGeometry g = logits_geometry(la.logits, la.dt, la.R, la.V, la.ld, la.beta);
    LocateParams lp;
    lp.f.logits = la.logits; lp.f.V = la.V; lp.f.ld = la.ld; lp.f.span = g.span; lp.f.n_spans = g.n_spans;
    lp.f.partials = reinterpret_cast<const float4*>(la.scratch); lp.f.beta = la.beta; lp.f.alpha_t = sa.alpha_t;
    lp.f.bf = g.bf; lp.f.vec = g.vec;
    lp.all = sa.all_triples; lp.P = sa.P; lp.rank = sa.rank; lp.R = la.R; lp.N = sa.N; lp.t = sa.t; lp.v0 = sa.v0;
    lp.tile_width = sa.tile_width;
    lp.seed = sa.seed; lp.done = la.done; lp.picks = sa.picks_out;
    auto fn = la.dt == PSMC_F32 ? pick_locate<PSMC_F32>(g.mode) : pick_locate<PSMC_BF16>(g.mode);
    return launch_chained(fn, dim3((unsigned)((la.R + kRowsPerCta - 1) / kRowsPerCta)), dim3(kRowsPerCta * 32), 0, stream,
                          lp);
}

cudaError_t launch_shard_owner_columns(const double* all_triples, int P, int R, int N, int t, double beta, uint64_t seed,
                                       const uint8_t* done, int tile_width, int32_t* need_out, cudaStream_t stream) {
    void (*fn)(const double*, int, int, int, int, double, uint64_t, const uint8_t*, int, int32_t*);
    switch (beta_mode(beta)) {
        case kBeta1: fn = shard_owner_columns_kernel<kBeta1>; break;
        case kBeta2: fn = shard_owner_columns_kernel<kBeta2>; break;
        case kBeta4: fn = shard_owner_columns_kernel<kBeta4>; break;
        case kBeta8: fn = shard_owner_columns_kernel<kBeta8>; break;
        default: fn = shard_owner_columns_kernel<kBetaAny>; break;
    }
    return launch_chained(fn, dim3((unsigned)((R + 255) / 256)), dim3(256), 0, stream, all_triples, P, R, N, t, beta, seed,
                          done, tile_width, need_out);
}

cudaError_t launch_shard_weights(const WeightsArgs& a, const double* all_triples, const psmc_shard_pick* all_picks, int P,
                                 cudaStream_t stream, bool picks_per_row) {
    ShardFinishParams sp;
    sp.a = a; sp.all = all_triples; sp.picks = all_picks; sp.P = P; sp.picks_per_row = picks_per_row ? 1 : 0;
    void (*fn)(const ShardFinishParams);
    switch (beta_mode(a.beta)) {
        case kBeta1: fn = shard_weights_kernel<kBeta1>; break;
        case kBeta2: fn = shard_weights_kernel<kBeta2>; break;
        case kBeta4: fn = shard_weights_kernel<kBeta4>; break;
        case kBeta8: fn = shard_weights_kernel<kBeta8>; break;
        default: fn = shard_weights_kernel<kBetaAny>; break;
    }
    const int warps = (a.N + 31) >> 5;
    const size_t stage_bytes = (size_t)a.N * P * 3 * sizeof(double);
    sp.staged = stage_bytes <= 4096 ? 1 : 0;  // (the static scratch of the group update takes most of the 48 KB)
    return launch_chained(fn, dim3((unsigned)a.G), dim3((unsigned)(warps * 32)), sp.staged ? stage_bytes : 0, stream, sp);
}

}  // namespace psmc
