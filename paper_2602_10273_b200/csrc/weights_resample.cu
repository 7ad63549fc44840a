// Second kernel of the step when it runs as two kernels: per-row finish of the logit pass (logits_common.cuh), then
// the per-group update of weights_core.cuh.  One CTA per group.
//
// Phase 1 (finish_rows: up to eight warps per particle, the CTA's warps shared among the group's rows):
// the span triples of the streaming kernel become the drawn token y, log p(y) and log omega of each row.
// Phase 2 (one thread per particle, N <= 1024; warp 0 alone when N <= 32): group_update().
#include "internal.h"
#include "logits_common.cuh"
#include "weights_core.cuh"

namespace psmc {
namespace {

struct KernelArgs {
    WeightsArgs a;
    FinishParams f;
    int wpr;  // warps per row in the finish
};

template <int DT, int MODE>
__global__ void __launch_bounds__(1024) finish_weights_resample_kernel(const __grid_constant__ KernelArgs ka) {
    __shared__ GroupScratch<kMaxParticles> sc;
    __shared__ FinishShared sh_fin;

    const WeightsArgs& a = ka.a;
    const int g = blockIdx.x, i = threadIdx.x, N = a.N;

    chain_begin();
    // the particles' state is asked for now and used after phase 1: its latency hides behind the row finishes
    ParticleState st{};
    if (i < N) st = load_particle(a, g * N + i);
    // ---- phase 1: the CTA's warps finish the rows of the group's live particles ----
    finish_rows<DT, MODE>(
        ka.f, sh_fin, g * N, N, ka.wpr, [&](int k) { return a.done[g * N + k] == 0; },
        [&](int k) { return hash_uniform(hash5(a.seed, kStreamToken, (uint64_t)g, (uint64_t)a.t, (uint64_t)k)); },
        [&](int k, const RowResult& rr) {
            if (rr.tok < 0) raise_status(a.status, PSMC_E_NUMERIC);
            sc.tok[k] = rr.tok;
            sc.S[k] = rr.logp;
            sc.C[k] = rr.loginc;
        });
    // finish_rows ends on a CTA-wide barrier: the results are visible to every thread

    // ---- phase 2: per-particle update ----
    const int nw = (N + 31) >> 5;  // warps that hold particles
    if (nw == 1 && i >= 32) return;  // up to 32 particles: warp 0 finishes alone, on warp collectives only
    const bool on = i < N;
    group_update(a, g, i, nw, sc, on ? sc.tok[i] : -1, on ? sc.S[i] : 0.0, on ? sc.C[i] : 0.0, st);
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
