// The logit pass as kernels of its own: the streaming sweep (logits_stream.cuh) followed by the per-row finish
// (logits_common.cuh).  Used by the stateless entry points and by the step when it cannot run as one fused kernel.
#include <mutex>

#include "logits_stream.cuh"

namespace psmc {
namespace {

// Rows that start on 16-byte boundaries.  Each warp owns a contiguous share of the (row, span) tasks, so it mostly
// stays inside one row and its copies walk forward through memory.
template <int DT, int MODE>
__global__ void __launch_bounds__(kMaxWarps * 32, 1) logits_stream_kernel(const __grid_constant__ StreamParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t bars[kMaxWarps * kDepth];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps_per_cta = blockDim.x >> 5;
    const int n_tasks = p.R * p.n_spans;  // < 2^31, checked by the host
    // Even shares: the tasks are dealt to the CTAs in contiguous runs that differ by at most one task, and a CTA's run
    // to its warps likewise.  (Rounding the share up per warp instead leaves whole SMs without work: 24 warps of 5 spans
    // cover 512 x 32 spans with 136 CTAs.)
    const int cta_base = n_tasks / (int)gridDim.x, cta_extra = n_tasks % (int)gridDim.x;
    const int cta_first = (int)blockIdx.x * cta_base + min((int)blockIdx.x, cta_extra);
    const int cta_n = cta_base + ((int)blockIdx.x < cta_extra ? 1 : 0);
    const int w_base = cta_n / warps_per_cta, w_extra = cta_n % warps_per_cta;
    const int first = cta_first + warp * w_base + min(warp, w_extra);
    const int per_warp = w_base + (warp < w_extra ? 1 : 0);
    const int last = first + per_warp;

    stream_init_barriers(bars + warp * kDepth, lane);
    chain_begin();  // everything above is local set-up; global memory from here on
    if (p.zero_words && blockIdx.x == 0 && threadIdx.x < 2) p.zero_words[threadIdx.x] = 0;
    stream_tasks<DT, MODE>(p, smem + (size_t)warp * kDepth * kStageBytes, bars + warp * kDepth, lane, first, last,
                           per_warp > 0 ? per_warp : 1, 0, [](int) {});
}

// Rows of any alignment: plain loads, 16 bytes per lane between a span's first and last 16-byte boundary.
template <int DT, int MODE>
__global__ void __launch_bounds__(256) logits_stream_scalar_kernel(const __grid_constant__ StreamParams p) {
    const int lane = threadIdx.x & 31;
    const int warp_global = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int n_warps = gridDim.x * (blockDim.x >> 5);
    if (p.zero_words && blockIdx.x == 0 && threadIdx.x < 2) p.zero_words[threadIdx.x] = 0;
    const PackedConsts kc = packed_consts(p.bf);
    const int n_tasks = p.R * p.n_spans;
    for (int task = warp_global; task < n_tasks; task += n_warps) {
        const int row = task / p.n_spans, sp = task - row * p.n_spans;
        if (p.done && p.done[row]) continue;
        const int a0 = sp * p.span, b0 = min(p.V, a0 + p.span);
        const void* rowp = reinterpret_cast<const char*>(p.logits) + (size_t)row * p.ld * (DT == PSMC_F32 ? 4 : 2);
        LaneSums acc = lane_sums_init();
        span_any_alignment<DT, MODE>(rowp, a0, b0, kc, lane, acc);
        store_triple<MODE>(p, row, sp, acc, lane);
    }
}

// the finish as a kernel of its own (stateless entry points): kFinishRows rows per CTA, four warps each
constexpr int kFinishRows = 8;
struct FinishKernelParams {
    FinishParams f;
    int R;
    const double* u;
    const uint8_t* done;
    int32_t* tok;
    double* logp;
    double* loginc;
    int32_t* status;
};
template <int DT, int MODE>
__global__ void __launch_bounds__(1024) logits_finish_kernel(const __grid_constant__ FinishKernelParams p) {
    __shared__ FinishShared sh;
    const int row0 = blockIdx.x * kFinishRows;
    const int n_rows = min(kFinishRows, p.R - row0);
    const int wpr = finish_warps_per_row(kFinishRows, p.f.span, blockDim.x >> 5);
    finish_rows<DT, MODE>(
        p.f, sh, row0, n_rows, wpr, [&](int k) { return !(p.done && p.done[row0 + k]); },
        [&](int k) { return p.u[row0 + k]; },
        [&](int k, const RowResult& r) {
            if (r.tok < 0) raise_status(p.status, PSMC_E_NUMERIC);
            p.tok[row0 + k] = r.tok;
            p.logp[row0 + k] = r.logp;
            p.loginc[row0 + k] = r.loginc;
        });
}

typedef void (*StreamFn)(const StreamParams);
template <int DT, bool VEC>
StreamFn pick_stream(int mode) {
    if (VEC) {
        switch (mode) {
            case kBeta1: return logits_stream_kernel<DT, kBeta1>;
            case kBeta2: return logits_stream_kernel<DT, kBeta2>;
            case kBeta4: return logits_stream_kernel<DT, kBeta4>;
            case kBeta8: return logits_stream_kernel<DT, kBeta8>;
            default: return logits_stream_kernel<DT, kBetaAny>;
        }
    }
    switch (mode) {
        case kBeta1: return logits_stream_scalar_kernel<DT, kBeta1>;
        case kBeta2: return logits_stream_scalar_kernel<DT, kBeta2>;
        case kBeta4: return logits_stream_scalar_kernel<DT, kBeta4>;
        case kBeta8: return logits_stream_scalar_kernel<DT, kBeta8>;
        default: return logits_stream_scalar_kernel<DT, kBetaAny>;
    }
}
typedef void (*FinishFn)(const FinishKernelParams);
template <int DT>
FinishFn pick_finish(int mode) {
    switch (mode) {
        case kBeta1: return logits_finish_kernel<DT, kBeta1>;
        case kBeta2: return logits_finish_kernel<DT, kBeta2>;
        case kBeta4: return logits_finish_kernel<DT, kBeta4>;
        case kBeta8: return logits_finish_kernel<DT, kBeta8>;
        default: return logits_finish_kernel<DT, kBetaAny>;
    }
}

}  // namespace

int logits_pass_span(int R, int V) {
    // about four spans per resident warp when the problem is large enough, between 1024 and 4096 logits each
    const int64_t resident_warps = (int64_t)kSMs * kMaxWarps;
    const int64_t want = ((int64_t)R * V) / (resident_warps * 4);
    int span = 1024;
    while (span < 4096 && span * 2 <= want) span *= 2;
    return span;
}

size_t logits_pass_scratch_bytes(int R, int V) {
    const int span = logits_pass_span(R, V);
    const size_t n_spans = ((size_t)V + span - 1) / span;
    return (size_t)R * n_spans * sizeof(float4);
}

LogitsGeometry logits_geometry(const void* logits, int dt, int R, int V, int64_t ld, double beta) {
    LogitsGeometry g;
    g.span = logits_pass_span(R, V);
    g.n_spans = (V + g.span - 1) / g.span;
    g.mode = beta_mode(beta);
    g.bf = (float)beta;
    const size_t esize = dt == PSMC_F32 ? 4 : 2;
    g.vec = (reinterpret_cast<uintptr_t>(logits) % 16 == 0) && ((ld * esize) % 16 == 0) ? 1 : 0;
    return g;
}

cudaError_t launch_logits_stream(const LogitsStreamArgs& a, cudaStream_t stream) {
    const LogitsGeometry g = logits_geometry(a.logits, a.dt, a.R, a.V, a.ld, a.beta);
    StreamParams p;
    p.logits = a.logits; p.R = a.R; p.V = a.V; p.ld = a.ld; p.span = g.span; p.n_spans = g.n_spans; p.bf = g.bf;
    p.done = a.done; p.partials = reinterpret_cast<float4*>(a.scratch); p.zero_words = a.zero_words;
    p.status = a.status;
    StreamFn fn;
    if (a.dt == PSMC_F32) fn = g.vec ? pick_stream<PSMC_F32, true>(g.mode) : pick_stream<PSMC_F32, false>(g.mode);
    else fn = g.vec ? pick_stream<PSMC_BF16, true>(g.mode) : pick_stream<PSMC_BF16, false>(g.mode);
    const int64_t n_tasks = (int64_t)a.R * g.n_spans;
    if (n_tasks >= (int64_t)1 << 31) return cudaErrorInvalidValue;
    if (!g.vec) {
        int64_t blocks = (n_tasks + 7) / 8;
        if (blocks > (int64_t)kSMs * 8) blocks = (int64_t)kSMs * 8;
        fn<<<(unsigned)(blocks < 1 ? 1 : blocks), 256, 0, stream>>>(p);
        return cudaGetLastError();
    }
    // one CTA per SM; as many warps per CTA as it takes to give every task a warp, up to kMaxWarps
    int64_t warps = (n_tasks + kSMs - 1) / kSMs;
    if (warps > kMaxWarps) warps = kMaxWarps;
    if (warps < 1) warps = 1;
    int64_t blocks = (n_tasks + warps - 1) / warps;
    if (blocks > kSMs) blocks = kSMs;
    const size_t smem = (size_t)warps * kDepth * kStageBytes;
    cudaError_t e = allow_dynamic_smem(reinterpret_cast<const void*>(fn), kMaxWarps * kDepth * kStageBytes);
    if (e != cudaSuccess) return e;
    return launch_chained(fn, dim3((unsigned)blocks), dim3((unsigned)(warps * 32)), smem, stream, p);
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
    using namespace psmc;
    if (!logits || !u || !scratch || !tok || !logp || !loginc || !status_word) return PSMC_E_INVAL;
    if (R < 1 || V < 2 || ld < V || !(beta > 0.0) || !(alpha_t >= 1.0)) return PSMC_E_INVAL;
    if (dt != PSMC_F32 && dt != PSMC_BF16) return PSMC_E_INVAL;
    if (scratch_bytes < logits_pass_scratch_bytes(R, V) || reinterpret_cast<uintptr_t>(scratch) % 256 != 0)
        return PSMC_E_INVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    LogitsStreamArgs a{};
    a.logits = logits; a.dt = dt; a.R = R; a.V = V; a.ld = ld; a.beta = beta; a.done = done; a.scratch = scratch;
    a.zero_words = nullptr;
    a.status = status_word;
    if (launch_logits_stream(a, s) != cudaSuccess) return PSMC_E_CUDA;

    const LogitsGeometry g = logits_geometry(logits, dt, R, V, ld, beta);
    FinishKernelParams p;
    p.f.logits = logits; p.f.V = V; p.f.ld = ld; p.f.span = g.span; p.f.n_spans = g.n_spans;
    p.f.partials = reinterpret_cast<const float4*>(scratch); p.f.beta = beta; p.f.alpha_t = alpha_t; p.f.bf = g.bf;
    p.f.vec = g.vec;
    p.R = R; p.u = u; p.done = done; p.tok = tok; p.logp = logp; p.loginc = loginc; p.status = status_word;
    FinishFn fn = dt == PSMC_F32 ? pick_finish<PSMC_F32>(g.mode) : pick_finish<PSMC_BF16>(g.mode);
    fn<<<(unsigned)((R + kFinishRows - 1) / kFinishRows), 1024, 0, s>>>(p);
    return cudaGetLastError() == cudaSuccess ? PSMC_OK : PSMC_E_CUDA;
}

// ---------------------------------------------------------------------------------------------
// The logit pass for callers that must not allocate: same two kernels, span triples kept in a
// fixed array that lives in the library's device image instead of in caller memory.
// ---------------------------------------------------------------------------------------------
namespace {

// Fixed scratch: room for PSMC_STATIC_SCRATCH_BYTES / 16 span triples.  It is part of the module, so
// every GPU on which the library gets loaded carries these 4 MiB until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[PSMC_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void* g_static_ptr[kMaxDevices];  // device address of g_static_scratch, looked up once per device

// `g_static_scratch` names a host-side handle in host code, not memory a kernel could use; the address
// the kernels need comes from the runtime, per device, with that device current.
cudaError_t static_scratch_address(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_static_ptr[dev] = ptr;
    }
    *out = g_static_ptr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" psmc_status psmc_logits_pass_static(const void* logits, psmc_dtype dt, int R, int V, int64_t ld,
                                               double beta, double alpha_t, const double* u, const uint8_t* done,
                                               int32_t* tok, double* logp, double* loginc, int32_t* status_word,
                                               void* stream) {
    using namespace psmc;
    if (!logits || !u || !tok || !logp || !loginc || !status_word) return PSMC_E_INVAL;
    if (R < 1 || V < 2 || ld < V || !(beta > 0.0) || !(alpha_t >= 1.0)) return PSMC_E_INVAL;
    if (dt != PSMC_F32 && dt != PSMC_BF16) return PSMC_E_INVAL;
    if (logits_pass_scratch_bytes(R, V) > (size_t)PSMC_STATIC_SCRATCH_BYTES) return PSMC_E_TOO_LARGE;
    void* scratch = nullptr;
    if (static_scratch_address(&scratch) != cudaSuccess) return PSMC_E_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // Nothing in the array has to start at zero: the streaming kernel writes every triple the finishing
    // kernel reads, so whatever an earlier call left behind is never looked at.
    LogitsStreamArgs a{};
    a.logits = logits; a.dt = dt; a.R = R; a.V = V; a.ld = ld; a.beta = beta; a.done = done; a.scratch = scratch;
    a.zero_words = nullptr;
    a.status = status_word;
    if (launch_logits_stream(a, s) != cudaSuccess) return PSMC_E_CUDA;

    const LogitsGeometry g = logits_geometry(logits, dt, R, V, ld, beta);
    FinishKernelParams p;
    p.f.logits = logits; p.f.V = V; p.f.ld = ld; p.f.span = g.span; p.f.n_spans = g.n_spans;
    p.f.partials = reinterpret_cast<const float4*>(scratch); p.f.beta = beta; p.f.alpha_t = alpha_t; p.f.bf = g.bf;
    p.f.vec = g.vec;
    p.R = R; p.u = u; p.done = done; p.tok = tok; p.logp = logp; p.loginc = loginc; p.status = status_word;
    FinishFn fn = dt == PSMC_F32 ? pick_finish<PSMC_F32>(g.mode) : pick_finish<PSMC_BF16>(g.mode);
    fn<<<(unsigned)((R + kFinishRows - 1) / kFinishRows), 1024, 0, s>>>(p);
    return cudaGetLastError() == cudaSuccess ? PSMC_OK : PSMC_E_CUDA;
}
