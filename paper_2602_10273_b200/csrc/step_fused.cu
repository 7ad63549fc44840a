// The whole per-token step as ONE kernel (groups of up to 32 particles, 16-byte aligned rows): the loop body of
// Algorithm 1 without the cache move.
//
// Every CTA (one per SM) runs up to kStreamers streaming warps (logits_stream.cuh) plus kFinishers finishing warps.
// The streaming warps take the (row, span) tasks of the logit block in short runs dealt round-robin over the whole
// grid, so the rows of the block complete one after the other while the sweep is still going on; after a span's
// triple is stored its warp counts one arrival for the row.  Finishing warp f owns rows f, f + F, ... in that
// order: it waits (bounded) until a row has all its arrivals, draws the row's token and Eq. 7 from the triples
// (finish_row_warp), and counts one arrival for the row's group; finished rows (absorbing EOS) arrive at once.
// The warp that brings a group to N arrivals runs the group's update (weights_core.cuh) on the spot.  Only the rows
// of the last wave and the last groups are finished after the sweep has ended; everything else hides behind it.
// The context uses this kernel for small logit blocks, where saving a launch matters most (step_can_fuse).
//
// The arrival counters are left at zero by their last user, so consecutive launches need no clearing.  The two
// counters of the move lists alternate between steps (the kernel clears the pair the next step will use), because
// a group may close and append to the lists while other CTAs are only starting.
#include <mutex>

#include "logits_stream.cuh"
#include "weights_core.cuh"

namespace psmc {
namespace {

constexpr int kFinishers = 2;            // finishing warps per CTA
constexpr int kStreamers = 16;           // streaming warps per CTA at most (small blocks: more would only sit idle)
constexpr int kRun = 2;                  // consecutive spans a streaming warp takes at a time
constexpr uint32_t kPollLimit = 1u << 19;  // polls of ~0.25 us before a finishing warp gives up on a row
constexpr int64_t kFuseMaxBytes = 8 << 20;  // logit blocks up to this size take the one-kernel step

struct FusedParams {
    StreamParams s;
    FinishParams f;
    WeightsArgs a;
    int32_t* row_arrivals;    // [R] spans of the row whose triple is stored
    int32_t* group_arrivals;  // [G] rows of the group that are finished
};

__device__ __forceinline__ int load_volatile(const int32_t* p) { return *reinterpret_cast<const volatile int32_t*>(p); }

template <int DT, int MODE>
__device__ __forceinline__ void finishing_warp(const FusedParams& fp, int fin_id, int n_fin, int lane, GroupScratch<32>& sc) {
    const WeightsArgs& a = fp.a;
    const int N = a.N;
    for (int row = fin_id; row < a.R; row += n_fin) {
        const int g = row / N, k = row - g * N;
        if (!a.done[row]) {
            int ok = 1;
            if (lane == 0) {
                uint32_t polls = 0;
                while (load_volatile(&fp.row_arrivals[row]) < fp.s.n_spans) {
                    if (++polls > kPollLimit) {
                        ok = 0;
                        break;
                    }
                    __nanosleep(256);
                }
                if (ok) fp.row_arrivals[row] = 0;  // every producer of this row has arrived: ready for the next launch
            }
            ok = __shfl_sync(kFull, ok, 0);
            __threadfence();  // the triples counted above are visible from here on
            RowResult rr{-1, 0.0, 0.0};
            if (ok) {
                const double U = hash_uniform(hash5(a.seed, kStreamToken, (uint64_t)g, (uint64_t)a.t, (uint64_t)k));
                rr = finish_row_warp<DT, MODE>(fp.f, row, U, lane);
            }
            if (lane == 0) {
                if (!ok) raise_status(a.status, PSMC_E_TIMEOUT);
                else if (rr.tok < 0) raise_status(a.status, PSMC_E_NUMERIC);
                a.tok[row] = rr.tok;
                a.logp[row] = rr.logp;
                a.loginc[row] = rr.loginc;
                __threadfence();
            }
        }
        int ticket = 0;
        if (lane == 0) ticket = atomicAdd(&fp.group_arrivals[g], 1);
        ticket = __shfl_sync(kFull, ticket, 0);
        if (ticket == N - 1) {  // the group is complete: this warp updates it
            if (lane == 0) fp.group_arrivals[g] = 0;
            __threadfence();
            int tk = -1;
            double lp = 0.0, inc = 0.0;
            ParticleState st{};
            if (lane < N) {
                const int r = g * N + lane;
                st = load_particle(a, r);
                tk = __ldcg(const_cast<const int32_t*>(a.tok) + r);
                lp = __ldcg(const_cast<const double*>(a.logp) + r);
                inc = __ldcg(const_cast<const double*>(a.loginc) + r);
            }
            group_update(a, g, lane, 1, sc, tk, lp, inc, st);
            __syncwarp();  // sc is reused by the next group this warp closes
        }
    }
}

template <int DT, int MODE>
__global__ void __launch_bounds__((kStreamers + kFinishers) * 32, 1) psmc_step_kernel(const __grid_constant__ FusedParams fp) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t bars[kStreamers * kDepth];
    __shared__ GroupScratch<32> sc[kFinishers];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n_stream = (blockDim.x >> 5) - kFinishers;  // streaming warps of this CTA
    if (warp < n_stream) {
        const StreamParams& p = fp.s;
        const int warp_global = blockIdx.x * n_stream + warp;
        const int n_warps = gridDim.x * n_stream;
        const int n_tasks = p.R * p.n_spans;  // < 2^31, checked by the host
        stream_init_barriers(bars + warp * kDepth, lane);
        chain_begin();  // everything above is local set-up; global memory from here on
        if (p.zero_words && blockIdx.x == 0 && threadIdx.x < 2) p.zero_words[threadIdx.x] = 0;
        stream_tasks<DT, MODE>(p, smem + (size_t)warp * kDepth * kStageBytes, bars + warp * kDepth, lane,
                               min(n_tasks, warp_global * kRun), n_tasks, kRun, (n_warps - 1) * kRun, [&](int row) {
                                   if (lane == 0) {
                                       __threadfence();  // the triple first, then the arrival
                                       atomicAdd(&fp.row_arrivals[row], 1);
                                   }
                               });
    } else {
        chain_begin();
        finishing_warp<DT, MODE>(fp, blockIdx.x * kFinishers + (warp - n_stream), gridDim.x * kFinishers, lane,
                                 sc[warp - n_stream]);
    }
}

typedef void (*FusedFn)(const FusedParams);
template <int DT>
FusedFn pick_fused(int mode) {
    switch (mode) {
        case kBeta1: return psmc_step_kernel<DT, kBeta1>;
        case kBeta2: return psmc_step_kernel<DT, kBeta2>;
        case kBeta4: return psmc_step_kernel<DT, kBeta4>;
        case kBeta8: return psmc_step_kernel<DT, kBeta8>;
        default: return psmc_step_kernel<DT, kBetaAny>;
    }
}

}  // namespace

// Measured on B200: with logit blocks of a few MB the step is bound by launch and dependency latency and one launch
// beats two (20-22 us against 26-28 us for 8 x 32000 and 16 x 151936 bf16 logits); from about 10 MB on, the tail of
// one-warp row finishes after the sweep costs more than the second kernel's 32 warps per group (58 us against 44 us
// for 512 x 128256).
bool step_can_fuse(const LogitsStreamArgs& la, int N) {
    const LogitsGeometry g = logits_geometry(la.logits, la.dt, la.R, la.V, la.ld, la.beta);
    const int64_t bytes = (int64_t)la.R * la.V * (la.dt == PSMC_F32 ? 4 : 2);
    return N <= 32 && g.vec != 0 && bytes <= kFuseMaxBytes;
}

cudaError_t launch_step_fused(const LogitsStreamArgs& la, const WeightsArgs& wa, int32_t* row_arrivals,
                              int32_t* group_arrivals, cudaStream_t stream) {
    const LogitsGeometry g = logits_geometry(la.logits, la.dt, la.R, la.V, la.ld, la.beta);
    const int64_t n_tasks = (int64_t)la.R * g.n_spans;
    if (n_tasks >= (int64_t)1 << 31) return cudaErrorInvalidValue;
    FusedParams fp;
    fp.s.logits = la.logits; fp.s.R = la.R; fp.s.V = la.V; fp.s.ld = la.ld; fp.s.span = g.span; fp.s.n_spans = g.n_spans;
    fp.s.bf = g.bf; fp.s.done = la.done; fp.s.partials = reinterpret_cast<float4*>(la.scratch);
    fp.s.zero_words = la.zero_words; fp.s.status = la.status;
    fp.f.logits = la.logits; fp.f.V = la.V; fp.f.ld = la.ld; fp.f.span = g.span; fp.f.n_spans = g.n_spans;
    fp.f.partials = reinterpret_cast<const float4*>(la.scratch); fp.f.beta = wa.beta; fp.f.alpha_t = wa.alpha_t;
    fp.f.bf = g.bf; fp.f.vec = g.vec;
    fp.a = wa;
    fp.row_arrivals = row_arrivals;
    fp.group_arrivals = group_arrivals;

    // one CTA per SM; as many streaming warps per CTA as it takes to give every run of spans a warp, up to kStreamers
    const int64_t units = (n_tasks + kRun - 1) / kRun;
    int64_t warps = (units + kSMs - 1) / kSMs;
    if (warps > kStreamers) warps = kStreamers;
    if (warps < 1) warps = 1;
    int64_t blocks = (units + warps - 1) / warps;
    if (blocks > kSMs) blocks = kSMs;
    const size_t smem = (size_t)warps * kDepth * kStageBytes;
    FusedFn fn = la.dt == PSMC_F32 ? pick_fused<PSMC_F32>(g.mode) : pick_fused<PSMC_BF16>(g.mode);
    cudaError_t e = allow_dynamic_smem(reinterpret_cast<const void*>(fn), kStreamers * kDepth * kStageBytes);
    if (e != cudaSuccess) return e;
    return launch_chained(fn, dim3((unsigned)blocks), dim3((unsigned)((warps + kFinishers) * 32)), smem, stream, fp);
}

}  // namespace psmc
