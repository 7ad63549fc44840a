// Streaming half of the logit pass: ONE sweep over the [R, V] logits, HBM-bound.
//
// A row is cut into spans of `span` consecutive logits; one warp streams one span with 128-bit
// loads (8 bf16 / 4 fp32 per lane per load, up to eight loads in flight per lane) and keeps, per
// lane, a running maximum m and the sums  s1 = sum exp(l - m),  sb = sum exp(beta (l - m)).
// One MUFU.EX2 per logit: for beta in {1,2,4,8} exp(beta d) is exp(d) squared up; other beta
// (exponent-bridging steps, Section 4.3) pay a second EX2.  The warp reduces its lanes to one
// (m, s1, sb) triple and stores it; nothing else leaves the kernel.  No atomics, no fences, no waits:
// spans are dealt round-robin to a grid that exactly fills the machine, so every warp does the same
// amount of work.  The per-row finish (logits_common.cuh) runs in the kernel that follows.
#include <mutex>

#include "internal.h"
#include "logits_common.cuh"

namespace psmc {
namespace {

constexpr int kThreads = 256;
constexpr int kWarpsPerCta = kThreads / 32;
constexpr int kCtasPerSm = 3;

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

struct LaneSums {
    float m, s1, sb;
};

// one logit into the two running sums; d = l - m
template <int MODE>
__device__ __forceinline__ void accumulate(float d, float cb, float& s1, float& sb) {
    const float e = ex2(d * kLog2e);
    s1 += e;
    if (MODE == kBeta2) {
        sb = fmaf(e, e, sb);
    } else if (MODE == kBeta4) {
        const float e2 = e * e;
        sb = fmaf(e2, e2, sb);
    } else if (MODE == kBeta8) {
        const float e2 = e * e;
        const float e4 = e2 * e2;
        sb = fmaf(e4, e4, sb);
    } else if (MODE == kBetaAny) {
        sb += ex2(d * cb);
    }
}
template <int MODE>
__device__ __forceinline__ void raise_max(float cm, float cb, LaneSums& a) {
    if (cm > a.m) {
        const float d0 = a.m - cm;  // <= 0; hugely negative on the first call, which zeroes the (empty) sums
        a.s1 *= ex2(d0 * kLog2e);
        if (MODE != kBeta1) a.sb *= mass_beta<MODE>(d0, cb);
        a.m = cm;
    }
}

// ---- bf16: NW 32-bit words = 2*NW logits ----
template <int MODE, int NW>
__device__ __forceinline__ void consume_bf16(const uint32_t (&w)[NW], float cb, LaneSums& a, __nv_bfloat162& m2) {
    __nv_bfloat162 pm = *reinterpret_cast<const __nv_bfloat162*>(&w[0]);
#pragma unroll
    for (int i = 1; i < NW; ++i) pm = __hmax2(pm, *reinterpret_cast<const __nv_bfloat162*>(&w[i]));
    if (!__hble2(pm, m2)) {  // some logit exceeds the running maximum (rare after the first loads)
        raise_max<MODE>(fmaxf(__low2float(pm), __high2float(pm)), cb, a);
        m2 = __float2bfloat162_rn(a.m);  // exact: m is itself a bf16 value
    }
#pragma unroll
    for (int i = 0; i < NW; ++i) {
        accumulate<MODE>(__uint_as_float(w[i] << 16) - a.m, cb, a.s1, a.sb);
        accumulate<MODE>(__uint_as_float(w[i] & 0xffff0000u) - a.m, cb, a.s1, a.sb);
    }
}
// ---- fp32: NW words = NW logits ----
template <int MODE, int NW>
__device__ __forceinline__ void consume_f32(const uint32_t (&w)[NW], float cb, LaneSums& a) {
    float cm = __uint_as_float(w[0]);
#pragma unroll
    for (int i = 1; i < NW; ++i) cm = fmaxf(cm, __uint_as_float(w[i]));
    raise_max<MODE>(cm, cb, a);
#pragma unroll
    for (int i = 0; i < NW; ++i) accumulate<MODE>(__uint_as_float(w[i]) - a.m, cb, a.s1, a.sb);
}
template <int DT, int MODE, int NW>
__device__ __forceinline__ void consume(const uint32_t (&w)[NW], float cb, LaneSums& a, __nv_bfloat162& m2) {
    if (DT == PSMC_BF16) consume_bf16<MODE, NW>(w, cb, a, m2);
    else consume_f32<MODE, NW>(w, cb, a);
}

// 16-byte aligned span [a0, b0) of a row: chunks of 16 bytes, lane-strided
template <int DT, int MODE>
__device__ __forceinline__ void span_vec(const void* rowp, int a0, int b0, float cb, int lane, LaneSums& acc) {
    constexpr int kPerChunk = DT == PSMC_BF16 ? 8 : 4;
    constexpr int kShift = DT == PSMC_BF16 ? 3 : 2;
    const int n = b0 - a0, n_chunks = n >> kShift;
    const uint4* p = reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(rowp) + (size_t)a0 * (16 / kPerChunk));
    __nv_bfloat162 m2 = __float2bfloat162_rn(acc.m);
    int c = lane;
    for (; c + 224 < n_chunks; c += 256) {  // eight loads in flight per lane
        uint4 v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = ld_stream16(p + c + 32 * i);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t w[16] = {v[4 * h].x,     v[4 * h].y,     v[4 * h].z,     v[4 * h].w,
                                    v[4 * h + 1].x, v[4 * h + 1].y, v[4 * h + 1].z, v[4 * h + 1].w,
                                    v[4 * h + 2].x, v[4 * h + 2].y, v[4 * h + 2].z, v[4 * h + 2].w,
                                    v[4 * h + 3].x, v[4 * h + 3].y, v[4 * h + 3].z, v[4 * h + 3].w};
            consume<DT, MODE, 16>(w, cb, acc, m2);
        }
    }
    for (; c + 96 < n_chunks; c += 128) {
        const uint4 v0 = ld_stream16(p + c), v1 = ld_stream16(p + c + 32), v2 = ld_stream16(p + c + 64),
                    v3 = ld_stream16(p + c + 96);
        const uint32_t w[16] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w,
                                v2.x, v2.y, v2.z, v2.w, v3.x, v3.y, v3.z, v3.w};
        consume<DT, MODE, 16>(w, cb, acc, m2);
    }
    for (; c < n_chunks; c += 32) {
        const uint4 v0 = ld_stream16(p + c);
        const uint32_t w[4] = {v0.x, v0.y, v0.z, v0.w};
        consume<DT, MODE, 4>(w, cb, acc, m2);
    }
    const int tail = n & (kPerChunk - 1);  // ragged end of the row
    if (lane < tail) {
        const float x = load_elem<DT>(rowp, (int64_t)a0 + (n_chunks << kShift) + lane);
        raise_max<MODE>(x, cb, acc);
        accumulate<MODE>(x - acc.m, cb, acc.s1, acc.sb);
    }
}

// any alignment: one logit per lane per load
template <int DT, int MODE>
__device__ __forceinline__ void span_scalar(const void* rowp, int a0, int b0, float cb, int lane, LaneSums& acc) {
    for (int i = a0 + lane; i < b0; i += 32) {
        const float x = load_elem<DT>(rowp, i);
        raise_max<MODE>(x, cb, acc);
        accumulate<MODE>(x - acc.m, cb, acc.s1, acc.sb);
    }
}

struct StreamParams {
    const void* logits;
    int R, V;
    int64_t ld;
    int span, n_spans;
    float cb;
    const uint8_t* done;
    float4* partials;
    int32_t* zero_words;
};

template <int DT, int MODE, bool VEC>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) logits_stream_kernel(const StreamParams p) {
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
        if (VEC) span_vec<DT, MODE>(rowp, a0, b0, p.cb, lane, acc);
        else span_scalar<DT, MODE>(rowp, a0, b0, p.cb, lane, acc);

        // one triple per span: rescale every lane to the warp's maximum, then add
        const float wm = warp_max(acc.m);
        const float d0 = acc.m - wm;
        float s1 = acc.s1 * ex2(d0 * kLog2e);
        float sb = (MODE == kBeta1) ? 0.f : acc.sb * mass_beta<MODE>(d0, p.cb);
        s1 = warp_sum(s1);
        sb = warp_sum(sb);
        if (lane == 0) __stcg(&p.partials[(size_t)row * p.n_spans + sp], make_float4(wm, s1, sb, 0.f));
    }
}

// one warp per row: the finish as a kernel of its own (stateless entry point)
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
__global__ void __launch_bounds__(kThreads) logits_finish_kernel(const FinishKernelParams p) {
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
    if (row >= p.R || (p.done && p.done[row])) return;
    const RowResult r = finish_row<DT, MODE>(p.f, row, p.u[row], lane);
    if (lane == 0) {
        if (r.tok < 0) raise_status(p.status, PSMC_E_NUMERIC);
        p.tok[row] = r.tok;
        p.logp[row] = r.logp;
        p.loginc[row] = r.loginc;
    }
}

typedef void (*StreamFn)(const StreamParams);
template <int DT, bool VEC>
StreamFn pick_stream(int mode) {
    switch (mode) {
        case kBeta1: return logits_stream_kernel<DT, kBeta1, VEC>;
        case kBeta2: return logits_stream_kernel<DT, kBeta2, VEC>;
        case kBeta4: return logits_stream_kernel<DT, kBeta4, VEC>;
        case kBeta8: return logits_stream_kernel<DT, kBeta8, VEC>;
        default: return logits_stream_kernel<DT, kBetaAny, VEC>;
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
    const int64_t resident_warps = (int64_t)kSMs * kCtasPerSm * kWarpsPerCta;
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
    g.cb = (float)(beta * 1.4426950408889634);
    const size_t esize = dt == PSMC_F32 ? 4 : 2;
    g.vec = (reinterpret_cast<uintptr_t>(logits) % 16 == 0) && ((ld * esize) % 16 == 0) ? 1 : 0;
    return g;
}

cudaError_t launch_logits_stream(const LogitsStreamArgs& a, cudaStream_t stream) {
    const LogitsGeometry g = logits_geometry(a.logits, a.dt, a.R, a.V, a.ld, a.beta);
    StreamParams p;
    p.logits = a.logits; p.R = a.R; p.V = a.V; p.ld = a.ld; p.span = g.span; p.n_spans = g.n_spans; p.cb = g.cb;
    p.done = a.done; p.partials = reinterpret_cast<float4*>(a.scratch); p.zero_words = a.zero_words;
    StreamFn fn;
    if (a.dt == PSMC_F32) fn = g.vec ? pick_stream<PSMC_F32, true>(g.mode) : pick_stream<PSMC_F32, false>(g.mode);
    else fn = g.vec ? pick_stream<PSMC_BF16, true>(g.mode) : pick_stream<PSMC_BF16, false>(g.mode);
    const int64_t n_tasks = (int64_t)a.R * g.n_spans;
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
    if (launch_logits_stream(a, s) != cudaSuccess) return PSMC_E_CUDA;

    const LogitsGeometry g = logits_geometry(logits, dt, R, V, ld, beta);
    FinishKernelParams p;
    p.f.logits = logits; p.f.V = V; p.f.ld = ld; p.f.span = g.span; p.f.n_spans = g.n_spans;
    p.f.partials = reinterpret_cast<const float4*>(scratch); p.f.beta = beta; p.f.alpha_t = alpha_t; p.f.cb = g.cb;
    p.f.vec = g.vec;
    p.R = R; p.u = u; p.done = done; p.tok = tok; p.logp = logp; p.loginc = loginc; p.status = status_word;
    FinishFn fn = dt == PSMC_F32 ? pick_finish<PSMC_F32>(g.mode) : pick_finish<PSMC_BF16>(g.mode);
    fn<<<(unsigned)((R + kWarpsPerCta - 1) / kWarpsPerCta), kThreads, 0, s>>>(p);
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
    if (launch_logits_stream(a, s) != cudaSuccess) return PSMC_E_CUDA;

    const LogitsGeometry g = logits_geometry(logits, dt, R, V, ld, beta);
    FinishKernelParams p;
    p.f.logits = logits; p.f.V = V; p.f.ld = ld; p.f.span = g.span; p.f.n_spans = g.n_spans;
    p.f.partials = reinterpret_cast<const float4*>(scratch); p.f.beta = beta; p.f.alpha_t = alpha_t; p.f.cb = g.cb;
    p.f.vec = g.vec;
    p.R = R; p.u = u; p.done = done; p.tok = tok; p.logp = logp; p.loginc = loginc; p.status = status_word;
    FinishFn fn = dt == PSMC_F32 ? pick_finish<PSMC_F32>(g.mode) : pick_finish<PSMC_BF16>(g.mode);
    fn<<<(unsigned)((R + kWarpsPerCta - 1) / kWarpsPerCta), kThreads, 0, s>>>(p);
    return cudaGetLastError() == cudaSuccess ? PSMC_OK : PSMC_E_CUDA;
}
