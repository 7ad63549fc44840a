// Streaming half of the logit pass: ONE sweep over the [R, V] logits, HBM-bound.
//
// A row is cut into spans of `span` consecutive logits; one warp sums one span and stores one (c, s1, sb)
// triple for it (logits_common.cuh); nothing else leaves the kernel.  The per-row finish runs in the kernel
// that follows.
//
// Data movement: one persistent CTA per SM, up to 16 warps, each warp with a private ring of kDepth stages of
// kStageBytes in shared memory.  Lane 0 of a warp keeps kDepth-1 bulk asynchronous copies (TMA, untiled,
// completion on an mbarrier) in flight for the pieces the warp will need next -- across span boundaries, so
// the memory pipe never drains -- while the warp sums the piece that has landed, reading it back with
// conflict-free 128-bit shared loads.  About 128 KB per SM are in flight at any time, independent of how the
// warps are scheduled.  No cross-warp synchronisation, no atomics; every mbarrier wait is bounded.
//
// Arithmetic per pair of logits: two unpack operations, two packed fp32x2 FMAs for x - c, two MUFU.EX2, one
// packed add for s1 and, for beta in {2,4,8}, one to three packed multiply/FMA for sb (2^{beta d} is 2^d
// squared up); other beta (exponent-bridging steps, Section 4.3) pay a second EX2 per logit.  The reference
// exponent c is common to the lanes of a warp and is carried from span to span inside a row.  It follows the
// largest logit the warp has seen with a slack of kRefSlack: it moves (a warp-uniform, rare path) only when some
// logit exceeds it by more than that, which keeps |x - c| of the dominant terms small -- the fp32 rounding of
// x - c is what limits their accuracy -- without rescaling the sums at every load.
#include <mutex>

#include "bulk_copy.cuh"
#include "internal.h"
#include "logits_common.cuh"

namespace psmc {
namespace {

constexpr int kMaxWarps = 16;        // warps per CTA of the streaming kernel
constexpr int kStageBytes = 4096;    // one bulk copy
constexpr int kDepth = 3;            // stages per warp: one being summed, two in flight
constexpr float kRefSlack = 2.0f;    // natural units a logit may exceed the warp's reference point by (less for beta > 31)

// ---- packed pairs of fp32 in one 64-bit register (fp32x2 instructions of sm_100) ----
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ float2 unpack2(f32x2 v) {
    float2 r;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(r.x), "=f"(r.y) : "l"(v));
    return r;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
// 2^x on both halves
__device__ __forceinline__ f32x2 ex2_2(f32x2 x) {
    f32x2 r;
    asm("{\n\t.reg .f32 lo, hi;\n\t"
        "mov.b64 {lo, hi}, %1;\n\t"
        "ex2.approx.ftz.f32 lo, lo;\n\t"
        "ex2.approx.ftz.f32 hi, hi;\n\t"
        "mov.b64 %0, {lo, hi};\n\t}"
        : "=l"(r)
        : "l"(x));
    return r;
}
// the two bf16 of a word, widened to fp32: low half in the low lane
__device__ __forceinline__ f32x2 widen_bf16x2(uint32_t w) {
    return ((f32x2)(w & 0xffff0000u) << 32) | (f32x2)(w << 16);
}

// Per-lane running state.  Two accumulators per sum (a, b) shorten the dependent chains; each holds a packed pair.
struct LaneSums {
    float thr;    // logits above this move the reference exponent (the same in every lane of the warp)
    float neg_c;  // minus the reference exponent in use (the same in every lane of the warp)
    f32x2 s1a, s1b, sba, sbb;
};
__device__ __forceinline__ LaneSums lane_sums_init() {
    LaneSums a;
    a.thr = kNegBig;
    a.neg_c = -kRefFloor;
    a.s1a = a.s1b = a.sba = a.sbb = 0ull;
    return a;
}
__device__ __forceinline__ float pair_sum(f32x2 v) {
    const float2 f = unpack2(v);
    return f.x + f.y;
}
__device__ __forceinline__ f32x2 pair_scale(f32x2 v, float f) { return mul2(v, pack2(f, f)); }

// The packed operations take no immediates; the constants they need live in registers for the whole kernel.
struct PackedConsts {
    f32x2 k_hi, k_lo, bf;
    float bf1;
    float slack;  // min(kRefSlack, 62 / beta): keeps 2^{beta slack log2 e} below 2^90
};
__device__ __forceinline__ PackedConsts packed_consts(float bf) {
    PackedConsts k;
    k.k_hi = pack2(kLog2eHi, kLog2eHi);
    k.k_lo = pack2(kLog2eLo, kLog2eLo);
    k.bf = pack2(bf, bf);
    k.bf1 = bf;
    k.slack = fminf(kRefSlack, 62.f / fmaxf(bf, 1.f));
    // hide the values from constant propagation so that they are not rebuilt at every use
    asm volatile("" : "+l"(k.k_hi), "+l"(k.k_lo), "+l"(k.bf));
    return k;
}
__device__ __forceinline__ f32x2 rel_exponent2(f32x2 l, f32x2 neg_c, const PackedConsts& k) {
    return fma2(l, k.k_lo, fma2(l, k.k_hi, neg_c));
}
// two logits, already as exponents d = x - c, into one accumulator pair
template <int MODE>
__device__ __forceinline__ void add_pair(f32x2 d, const PackedConsts& k, f32x2& s1, f32x2& sb) {
    const f32x2 e = ex2_2(d);
    s1 = add2(s1, e);
    if (MODE == kBeta2) {
        sb = fma2(e, e, sb);
    } else if (MODE == kBeta4) {
        const f32x2 e2 = mul2(e, e);
        sb = fma2(e2, e2, sb);
    } else if (MODE == kBeta8) {
        const f32x2 e2 = mul2(e, e);
        const f32x2 e4 = mul2(e2, e2);
        sb = fma2(e4, e4, sb);
    } else if (MODE == kBetaAny) {
        sb = add2(sb, ex2_2(mul2(d, k.bf)));
    }
}
// Some lane met a logit above the threshold; cm is this lane's largest candidate.  The warp moves its reference
// exponent to the largest of them and shrinks the sums accordingly.  Called by all 32 lanes together.
// Logits up to the new maximum + slack then pass without another move: a term stays below
// 2^{beta slack log2 e} <= 2^90 and whatever underflows is smaller than 2^-126 against a largest term of about 1.
template <int MODE>
__device__ __forceinline__ void move_reference(float cm, float bf, float slack, LaneSums& a) {
    cm = warp_max(cm);
    const float new_neg_c = -ref_exponent(cm);
    const float d0 = new_neg_c - a.neg_c;  // c_old - c_new < 0; hugely negative the first time, when the sums are empty
    const float f1 = ex2(d0);
    a.s1a = pair_scale(a.s1a, f1);
    a.s1b = pair_scale(a.s1b, f1);
    if (MODE != kBeta1) {
        const float fb = mass_beta<MODE>(d0, bf);
        a.sba = pair_scale(a.sba, fb);
        a.sbb = pair_scale(a.sbb, fb);
    }
    a.thr = cm + slack;
    a.neg_c = new_neg_c;
}
// one logit per lane (ragged ends, unaligned rows); all 32 lanes call it, lanes without a logit pass -inf
template <int MODE>
__device__ __forceinline__ void add_one(float l, float bf, float slack, LaneSums& a) {
    if (__any_sync(kFull, l > a.thr)) move_reference<MODE>(l, bf, slack, a);
    const float d = rel_exponent(l, a.neg_c);  // -inf for a lane without a logit: mass 0
    a.s1a = add2(a.s1a, pack2(ex2(d), 0.f));
    if (MODE != kBeta1) a.sba = add2(a.sba, pack2(mass_beta<MODE>(d, bf), 0.f));
}

// ---- bf16: NW 32-bit words = 2*NW logits ----
template <int MODE, int NW>
__device__ __forceinline__ void consume_bf16(const uint32_t (&w)[NW], const PackedConsts& k, LaneSums& a,
                                             __nv_bfloat162& thr2) {
    __nv_bfloat162 pm = *reinterpret_cast<const __nv_bfloat162*>(&w[0]);
#pragma unroll
    for (int i = 1; i < NW; ++i) pm = __hmax2(pm, *reinterpret_cast<const __nv_bfloat162*>(&w[i]));
    if (__any_sync(kFull, !__hble2(pm, thr2))) {  // some logit of the warp is above the threshold
        move_reference<MODE>(fmaxf(__low2float(pm), __high2float(pm)), k.bf1, k.slack, a);
        thr2 = __float2bfloat162_rn(a.thr);
    }
    const f32x2 nc = pack2(a.neg_c, a.neg_c);
#pragma unroll
    for (int i = 0; i < NW; ++i) {
        const f32x2 d = rel_exponent2(widen_bf16x2(w[i]), nc, k);
        if (i & 1) add_pair<MODE>(d, k, a.s1b, a.sbb);
        else add_pair<MODE>(d, k, a.s1a, a.sba);
    }
}
// ---- fp32: NW words = NW logits (NW even) ----
template <int MODE, int NW>
__device__ __forceinline__ void consume_f32(const uint32_t (&w)[NW], const PackedConsts& k, LaneSums& a) {
    float cm = __uint_as_float(w[0]);
#pragma unroll
    for (int i = 1; i < NW; ++i) cm = fmaxf(cm, __uint_as_float(w[i]));
    if (__any_sync(kFull, cm > a.thr)) move_reference<MODE>(cm, k.bf1, k.slack, a);
    const f32x2 nc = pack2(a.neg_c, a.neg_c);
#pragma unroll
    for (int i = 0; i < NW; i += 2) {
        const f32x2 d = rel_exponent2(((f32x2)w[i + 1] << 32) | (f32x2)w[i], nc, k);
        if (i & 2) add_pair<MODE>(d, k, a.s1b, a.sbb);
        else add_pair<MODE>(d, k, a.s1a, a.sba);
    }
}
template <int DT, int MODE, int NW>
__device__ __forceinline__ void consume(const uint32_t (&w)[NW], const PackedConsts& k, LaneSums& a,
                                        __nv_bfloat162& thr2) {
    if (DT == PSMC_BF16) consume_bf16<MODE, NW>(w, k, a, thr2);
    else consume_f32<MODE, NW>(w, k, a);
}

// any alignment: one logit per lane per load
template <int DT, int MODE>
__device__ __forceinline__ void span_scalar(const void* rowp, int a0, int b0, const PackedConsts& k, int lane,
                                            LaneSums& acc) {
    for (int i0 = a0; i0 < b0; i0 += 32)  // the same trip count in every lane
        add_one<MODE>(i0 + lane < b0 ? load_elem<DT>(rowp, i0 + lane) : -INFINITY, k.bf1, k.slack, acc);
}

struct StreamParams {
    const void* logits;
    int R, V;
    int64_t ld;
    int span, n_spans;
    float bf;     // (float)beta
    const uint8_t* done;
    float4* partials;
    int32_t* zero_words;
    int32_t* status;  // may be NULL
};

// one (row, span) task as the streaming loop sees it
struct TaskDesc {
    int row, sp;
    int bytes16;        // bytes of the span that bulk copies can fetch (a multiple of 16)
    int tail;           // ragged logits after them (only a row's last span can have any)
    const char* base;   // first byte of the span
};
// Walks the tasks first, first+1, ... in (row, span) order without dividing at every step.
template <int DT>
struct TaskWalker {
    int task, end, row, sp;
    __device__ __forceinline__ void start(const StreamParams& p, int first, int last) {
        task = first;
        end = last;
        row = first / p.n_spans;
        sp = first - row * p.n_spans;
    }
    __device__ __forceinline__ bool at_end() const { return task >= end; }
    __device__ __forceinline__ void next(const StreamParams& p) {
        ++task;
        if (++sp == p.n_spans) {
            sp = 0;
            ++row;
        }
    }
    // false: the row is finished and its logits are not to be read (absorbing state)
    __device__ __forceinline__ bool describe(const StreamParams& p, TaskDesc& d) const {
        constexpr int kPer = DT == PSMC_BF16 ? 8 : 4;  // logits per 16 bytes
        if (p.done && p.done[row]) return false;
        d.row = row;
        d.sp = sp;
        const int a0 = sp * p.span;
        const int n = min(p.V, a0 + p.span) - a0;
        d.bytes16 = (n / kPer) * 16;
        d.tail = n % kPer;
        d.base = reinterpret_cast<const char*>(p.logits) + ((size_t)row * p.ld + a0) * (16 / kPer);
        return true;
    }
};

// one triple per span: the lanes share the reference exponent, so their sums add up as they are
template <int MODE>
__device__ __forceinline__ void store_triple(const StreamParams& p, int row, int sp, const LaneSums& acc, int lane) {
    const float s1 = warp_sum(pair_sum(add2(acc.s1a, acc.s1b)));
    const float sb = (MODE == kBeta1) ? 0.f : warp_sum(pair_sum(add2(acc.sba, acc.sbb)));
    if (lane == 0) __stcg(&p.partials[(size_t)row * p.n_spans + sp], make_float4(-acc.neg_c, s1, sb, 0.f));
}

// Rows that start on 16-byte boundaries: the bulk-copy pipeline described at the top of the file.  Each warp owns
// a contiguous run of tasks, so it mostly stays inside one row and its copies walk forward through memory.
template <int DT, int MODE>
__global__ void __launch_bounds__(kMaxWarps * 32, 1) logits_stream_kernel(const __grid_constant__ StreamParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t bars[kMaxWarps * kDepth];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps_per_cta = blockDim.x >> 5;
    const int warp_global = blockIdx.x * warps_per_cta + warp;
    const int n_warps = gridDim.x * warps_per_cta;
    const int n_tasks = p.R * p.n_spans;  // < 2^31, checked by the host
    const int per_warp = (n_tasks + n_warps - 1) / n_warps;
    const int first = min(n_tasks, warp_global * per_warp), last = min(n_tasks, first + per_warp);

    const PackedConsts kc = packed_consts(p.bf);
    unsigned char* ring = smem + (size_t)warp * kDepth * kStageBytes;
    uint64_t* full = bars + warp * kDepth;
    if (lane == 0) {
        for (int d = 0; d < kDepth; ++d) mbar_init(&full[d], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    __syncwarp();
    chain_begin();  // everything above is local set-up; global memory from here on
    if (p.zero_words && blockIdx.x == 0 && threadIdx.x < 2) p.zero_words[threadIdx.x] = 0;

    // producer cursor (the same in every lane; lane 0 issues): the next piece to fetch
    TaskWalker<DT> pw;
    pw.start(p, first, last);
    const char* p_src = nullptr;
    int p_left = 0;
    auto prod_seek = [&]() {
        for (; !pw.at_end(); pw.next(p)) {
            TaskDesc d;
            if (pw.describe(p, d) && d.bytes16 > 0) {
                p_src = d.base;
                p_left = d.bytes16;
                return;
            }
        }
    };
    int issued = 0;
    auto issue = [&]() {  // next piece into stage issued % kDepth
        if (pw.at_end()) return;
        const int bytes = p_left < kStageBytes ? p_left : kStageBytes;
        if (lane == 0) {
            const int slot = issued % kDepth;
            fence_async_smem();  // the stage's previous contents were read through the generic proxy
            mbar_expect_tx(&full[slot], (uint32_t)bytes);
            bulk_load(ring + (size_t)slot * kStageBytes, p_src, (uint32_t)bytes, &full[slot]);
        }
        ++issued;
        p_src += bytes;
        p_left -= bytes;
        if (p_left == 0) {
            pw.next(p);
            prod_seek();
        }
    };

    // consumer cursor: the task being summed
    TaskWalker<DT> cw;
    cw.start(p, first, last);
    int c_left = 0, c_row = -1;
    TaskDesc c_d = {};
    LaneSums acc = lane_sums_init();
    __nv_bfloat162 thr2 = __float2bfloat162_rn(acc.thr);
    auto finish_task = [&]() {
        if (c_d.tail > 0)  // ragged end of the row
            add_one<MODE>(lane < c_d.tail ? load_elem<DT>(c_d.base + c_d.bytes16, lane) : -INFINITY, kc.bf1, kc.slack, acc);
        store_triple<MODE>(p, c_d.row, c_d.sp, acc, lane);
    };
    auto cons_seek = [&]() {  // next live task; tasks without a whole 16-byte chunk are done on the spot
        for (; !cw.at_end(); cw.next(p)) {
            if (cw.describe(p, c_d)) {
                if (c_d.row != c_row) {  // a new row: forget the reference point of the old one
                    acc = lane_sums_init();
                    thr2 = __float2bfloat162_rn(acc.thr);
                    c_row = c_d.row;
                } else {                 // same row: keep the reference point, start new sums
                    acc.s1a = acc.s1b = acc.sba = acc.sbb = 0ull;
                }
                c_left = c_d.bytes16;
                if (c_left > 0) return;
                finish_task();
            }
        }
    };

    prod_seek();
    cons_seek();
    for (int d = 0; d < kDepth - 1; ++d) issue();

    bool failed = false;
    int consumed = 0;
    while (!cw.at_end()) {
        __syncwarp();  // every lane is done with the stage that is about to be refilled
        issue();
        const int slot = consumed % kDepth;
        if (!__all_sync(kFull, mbar_wait(&full[slot], (uint32_t)((consumed / kDepth) & 1)))) {  // uniform verdict
            failed = true;
            break;
        }
        const uint4* st = reinterpret_cast<const uint4*>(ring + (size_t)slot * kStageBytes);
        const int bytes = c_left < kStageBytes ? c_left : kStageBytes;
        if (bytes == kStageBytes) {
#pragma unroll
            for (int h = 0; h < kStageBytes / 2048; ++h) {  // 2 KB = four 16-byte chunks per lane at a time
                const uint4 v0 = st[h * 128 + lane], v1 = st[h * 128 + 32 + lane], v2 = st[h * 128 + 64 + lane],
                            v3 = st[h * 128 + 96 + lane];
                const uint32_t w[16] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w,
                                        v2.x, v2.y, v2.z, v2.w, v3.x, v3.y, v3.z, v3.w};
                consume<DT, MODE, 16>(w, kc, acc, thr2);
            }
        } else {
            constexpr uint32_t kNoLogit = DT == PSMC_BF16 ? 0xff80ff80u : 0xff800000u;  // -inf: no mass, never a maximum
            for (int c0 = 0; c0 < (bytes >> 4); c0 += 32) {  // the same trip count in every lane
                const bool in = c0 + lane < (bytes >> 4);
                const uint4 v0 = in ? st[c0 + lane] : make_uint4(kNoLogit, kNoLogit, kNoLogit, kNoLogit);
                const uint32_t w[4] = {v0.x, v0.y, v0.z, v0.w};
                consume<DT, MODE, 4>(w, kc, acc, thr2);
            }
        }
        ++consumed;
        c_left -= bytes;
        if (c_left == 0) {
            finish_task();
            cw.next(p);
            cons_seek();
        }
    }
    if (failed) {
        if (lane == 0) raise_status(p.status, PSMC_E_TIMEOUT);
        // do not leave with copies still landing in this CTA's shared memory: bounded second wait
        for (int j = consumed; j < issued; ++j) mbar_wait(&full[j % kDepth], (uint32_t)((j / kDepth) & 1));
    }
}

// Rows of any alignment: plain loads, one logit per lane per load.
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
        span_scalar<DT, MODE>(rowp, a0, b0, kc, lane, acc);
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
    {
        static std::mutex mu;
        static bool configured[2][5] = {};
        std::lock_guard<std::mutex> lock(mu);
        if (!configured[a.dt][g.mode]) {
            cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 kMaxWarps * kDepth * kStageBytes);
            if (e != cudaSuccess) return e;
            configured[a.dt][g.mode] = true;
        }
    }
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
