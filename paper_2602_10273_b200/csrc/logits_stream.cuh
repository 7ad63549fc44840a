// Streaming half of the logit pass: ONE sweep over the [R, V] logits, HBM-bound.
//
// A row is cut into spans of `span` consecutive logits; one warp sums one span and stores one (c, s1, sb)
// triple for it (logits_common.cuh); nothing else leaves the kernel.  The per-row finish runs in the kernel
// that follows.
//
// Data movement: one persistent CTA per SM, up to kMaxWarps warps, each warp with a private ring of kDepth stages of
// kStageBytes in shared memory.  Lane 0 of a warp keeps kDepth-1 bulk asynchronous copies (TMA, untiled,
// completion on an mbarrier) in flight for the pieces the warp will need next -- across span boundaries, so
// the memory pipe never drains -- while the warp sums the piece that has landed, reading it back with
// conflict-free 128-bit shared loads.  With 24 warps and two stages of 4 KB each, about 96 KB per SM are in flight
// at any time, independent of how the warps are scheduled (a pure read of this shape runs no faster three deep, and
// 24 warps hide the latencies of the arithmetic better than 16: 31 us against 33 us for 512 x 128256 bf16 logits).
// No cross-warp synchronisation, no atomics; every mbarrier wait is bounded.
//
// Arithmetic per pair of logits: two unpack operations, two packed fp32x2 FMAs for x - c, two MUFU.EX2, one
// packed add for s1 and, for beta in {2,4,8}, one to three packed multiply/FMA for sb (2^{beta d} is 2^d
// squared up); other beta (exponent-bridging steps, Section 4.3) pay a second EX2 per logit.  The reference
// exponent c is common to the lanes of a warp and is carried from span to span inside a row.  It follows the
// largest logit the warp has seen with a slack of kRefSlack: it moves (a warp-uniform, rare path) only when some
// logit exceeds it by more than that, which keeps |x - c| of the dominant terms small -- the fp32 rounding of
// x - c is what limits their accuracy -- without rescaling the sums at every load.
#pragma once

#include "bulk_copy.cuh"
#include "internal.h"
#include "logits_common.cuh"

namespace psmc {

constexpr int kMaxWarps = 24;        // warps per CTA of the streaming kernel
constexpr int kStageBytes = 4096;    // one bulk copy
constexpr int kDepth = 2;            // stages per warp: one being summed, one in flight
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
// The warp's total of one sum, from the lanes' four partial sums each: added up in fp64 and rounded to fp32 once.
// (A partner below half an ulp of the partial sum that holds the row's dominant term would vanish in an fp32 tree,
// the remainders of compensated sums among them.)
__device__ __forceinline__ float warp_total(f32x2 a, f32x2 b) {
    const float2 fa = unpack2(a), fb = unpack2(b);
    const double t = ((double)fa.x + (double)fb.x) + ((double)fa.y + (double)fb.y);
    return (float)warp_sum(t);
}
__device__ __forceinline__ f32x2 pair_scale(f32x2 v, float f) { return mul2(v, pack2(f, f)); }

// The packed operations take no immediates; the constants they need live in registers for the whole kernel.
struct PackedConsts {
    f32x2 k_hi, k_lo, bf;
    float bf1;
    float slack;  // how far a logit may exceed the largest one seen before the reference moves (natural units)
    float shift;  // ref_shift(beta)
};
__device__ __forceinline__ PackedConsts packed_consts(float bf) {
    PackedConsts k;
    k.k_hi = pack2(kLog2eHi, kLog2eHi);
    k.k_lo = pack2(kLog2eLo, kLog2eLo);
    k.bf = pack2(bf, bf);
    k.bf1 = bf;
    k.shift = ref_shift(bf);
    // With the shift the largest term of a sum has an exponent between -2 - slack log2(e) and -1, and what limits the
    // accuracy of a term is the fp32 rounding of beta (x - c): the slack shrinks as beta grows, 4 / beta natural
    // units, so that beta |x - c| of the largest terms stays below 2 beta + 5.8.  (At beta = 4 a slack of 2 was
    // measured to break the ESS agreement with the oracle, 1e-6 N, on 512 x 128256 logits; 1 holds it.)  Without the
    // shift (large beta) the slack keeps 2^{beta (x - c)} in range.
    k.slack = k.shift != 0.f ? fminf(kRefSlack, 4.f / fmaxf(bf, 1.f)) : fminf(kRefSlack, 62.f / bf);
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
// exponent beyond the largest of them plus the slack and shrinks the sums accordingly.  Called by all 32 lanes
// together.  Logits up to the new maximum + slack then pass without another move; every term stays at or below 1/2,
// the largest ones lie between 2^{-2 - slack log2 e} and 1/2, and whatever underflows is smaller than 2^-120 of them.
template <int MODE>
__device__ __forceinline__ void move_reference(float cm, const PackedConsts& k, LaneSums& a) {
    const float bf = k.bf1, slack = k.slack;
    cm = warp_max(cm);
    // with the shift, logits up to the new threshold keep their exponents at or below -1
    const float new_neg_c = -(k.shift != 0.f ? ref_exponent(cm + slack, 1.f) : ref_exponent(cm, 0.f));
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
__device__ __forceinline__ void add_one(float l, const PackedConsts& k, LaneSums& a) {
    const float bf = k.bf1;
    if (__any_sync(kFull, l > a.thr)) move_reference<MODE>(l, k, a);
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
        move_reference<MODE>(fmaxf(__low2float(pm), __high2float(pm)), k, a);
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
    if (__any_sync(kFull, cm > a.thr)) move_reference<MODE>(cm, k, a);
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

// any alignment: one logit per lane per load.  A lane has one running sum here, not four, and the sum that holds a
// row's dominant term swallows every later term below half an ulp of it, always downwards (measured on rows with one
// token far above the rest: ln(sum) low by 2e-8 to 4e-8, the same at every token, which adds up in log p(y_{1:t})).
// So the sum of the 2^{x-c} is compensated: what each addition rounds away is collected in the second accumulator,
// which the warp's total adds back.
template <int DT, int MODE>
__device__ __forceinline__ void span_scalar(const void* rowp, int a0, int b0, const PackedConsts& k, int lane,
                                            LaneSums& acc) {
    for (int i0 = a0; i0 < b0; i0 += 32) {  // the same trip count in every lane
        const float l = i0 + lane < b0 ? load_elem<DT>(rowp, i0 + lane) : -INFINITY;
        if (__any_sync(kFull, l > acc.thr)) move_reference<MODE>(l, k, acc);  // (scales sum and remainder alike)
        const float d = rel_exponent(l, acc.neg_c);  // -inf for a lane without a logit: mass 0
        const float e = ex2(d);
        float2 s = unpack2(acc.s1a), r = unpack2(acc.s1b);
        const float t = s.x + e, virt = t - s.x;
        r.x += (s.x - (t - virt)) + (e - virt);  // exactly what the addition lost
        s.x = t;
        acc.s1a = pack2(s.x, s.y);
        acc.s1b = pack2(r.x, r.y);
        if (MODE != kBeta1) acc.sba = add2(acc.sba, pack2(mass_beta<MODE>(d, k.bf1), 0.f));
    }
}

// A span of a row that starts anywhere (rows whose pitch or base is not a multiple of 16 bytes: a vocabulary of odd
// size in a dense tensor).  The logits up to the first 16-byte boundary and after the last one go one per lane; the
// stretch between them is read 16 bytes per lane at a time and summed exactly as the staged sweep sums its stages.
template <int DT, int MODE>
__device__ __forceinline__ void span_any_alignment(const void* rowp, int a0, int b0, const PackedConsts& k, int lane,
                                                   LaneSums& acc) {
    constexpr int kEs = DT == PSMC_F32 ? 4 : 2, kPer = 16 / kEs;
    const uintptr_t addr = reinterpret_cast<uintptr_t>(rowp) + (size_t)a0 * kEs;
    int head = (addr % kEs) ? b0 - a0 : (int)(((16 - (addr & 15)) & 15) / kEs);  // (a base off its element size: all scalar)
    head = head < b0 - a0 ? head : b0 - a0;
    const int mid0 = a0 + head, chunks = (b0 - mid0) / kPer, tail0 = mid0 + chunks * kPer;
    if (head > 0) span_scalar<DT, MODE>(rowp, a0, mid0, k, lane, acc);
    if (chunks > 0) {
        __nv_bfloat162 thr2 = __float2bfloat162_rn(acc.thr);
        const uint4* q = reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(rowp) + (size_t)mid0 * kEs);
        int c0 = 0;
        for (; c0 + 128 <= chunks; c0 += 128) {  // four 16-byte loads per lane in flight
            const uint4 v0 = __ldg(&q[c0 + lane]), v1 = __ldg(&q[c0 + 32 + lane]), v2 = __ldg(&q[c0 + 64 + lane]),
                        v3 = __ldg(&q[c0 + 96 + lane]);
            const uint32_t w[16] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w,
                                    v2.x, v2.y, v2.z, v2.w, v3.x, v3.y, v3.z, v3.w};
            consume<DT, MODE, 16>(w, k, acc, thr2);
        }
        constexpr uint32_t kNoLogit = DT == PSMC_BF16 ? 0xff80ff80u : 0xff800000u;  // -inf: no mass, never a maximum
        for (; c0 < chunks; c0 += 32) {  // the same trip count in every lane
            const bool in = c0 + lane < chunks;
            const uint4 v0 = in ? __ldg(&q[c0 + lane]) : make_uint4(kNoLogit, kNoLogit, kNoLogit, kNoLogit);
            const uint32_t w[4] = {v0.x, v0.y, v0.z, v0.w};
            consume<DT, MODE, 4>(w, k, acc, thr2);
        }
    }
    if (tail0 < b0) span_scalar<DT, MODE>(rowp, tail0, b0, k, lane, acc);
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
// Walks a warp's tasks in (row, span) order: runs of `run` consecutive tasks, `skip` tasks apart, without dividing
// at every step.  One run covering everything gives a contiguous share; short runs dealt round-robin make the rows
// of the block complete one after the other.
template <int DT>
struct TaskWalker {
    int task, end, row, sp, run, run_left, skip;
    int flag_row;        // row whose finished flag is held in `flag` (-1: none yet)
    unsigned char flag;
    __device__ __forceinline__ void seat(const StreamParams& p) {
        row = task / p.n_spans;
        sp = task - row * p.n_spans;
    }
    __device__ __forceinline__ void start(const StreamParams& p, int first, int last, int run_len, int skip_len) {
        task = first;
        end = last;
        run = run_left = run_len;
        skip = skip_len;
        flag_row = -1;
        flag = 0;
        seat(p);
    }
    __device__ __forceinline__ bool at_end() const { return task >= end; }
    __device__ __forceinline__ void next(const StreamParams& p) {
        ++task;
        if (--run_left == 0) {
            run_left = run;
            task += skip;
            if (task < end) seat(p);
        } else if (++sp == p.n_spans) {
            sp = 0;
            ++row;
        }
    }
    // false: the row is finished and its logits are not to be read (absorbing state)
    __device__ __forceinline__ bool describe(const StreamParams& p, TaskDesc& d) {
        constexpr int kPer = DT == PSMC_BF16 ? 8 : 4;  // logits per 16 bytes
        if (row != flag_row) {  // one trip to memory per row, not per span: the warp waits for it with nothing in flight
            flag_row = row;
            flag = p.done ? p.done[row] : 0;
        }
        if (flag) return false;
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
    const float s1 = warp_total(acc.s1a, acc.s1b);
    const float sb = (MODE == kBeta1) ? 0.f : warp_total(acc.sba, acc.sbb);
    if (lane == 0) __stcg(&p.partials[(size_t)row * p.n_spans + sp], make_float4(-acc.neg_c, s1, sb, 0.f));
}
// The streaming loop of one warp (rows that start on 16-byte boundaries): the bulk-copy pipeline described at the top
// of the file over the tasks [first, last) taken in runs of `run` every `run + skip`.  ring: the warp's kDepth stages;
// full: its kDepth mbarriers, initialised; stored(row) is called by every lane after a span's triple went out.
// Returns false when a bounded wait ran out (the status word is set and the warp's copies have been drained).
template <int DT, int MODE, class StoredFn>
__device__ __forceinline__ bool stream_tasks(const StreamParams& p, unsigned char* ring, uint64_t* full, int lane, int first,
                                             int last, int run, int skip, StoredFn stored) {
    const PackedConsts kc = packed_consts(p.bf);

    // producer cursor (the same in every lane; lane 0 issues): the next piece to fetch
    TaskWalker<DT> pw;
    pw.start(p, first, last, run, skip);
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
    cw.start(p, first, last, run, skip);
    int c_left = 0, c_row = -1;
    TaskDesc c_d = {};
    LaneSums acc = lane_sums_init();
    __nv_bfloat162 thr2 = __float2bfloat162_rn(acc.thr);
    auto finish_task = [&]() {
        if (c_d.tail > 0)  // ragged end of the row
            add_one<MODE>(lane < c_d.tail ? load_elem<DT>(c_d.base + c_d.bytes16, lane) : -INFINITY, kc, acc);
        store_triple<MODE>(p, c_d.row, c_d.sp, acc, lane);
        stored(c_d.row);
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
        if (!__all_sync(kFull, mbar_wait(&full[slot], (uint32_t)((consumed / kDepth) & 1)))) {  // the same answer in every lane
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
    return !failed;
}

// set-up of a warp's mbarriers; every lane of the warp calls it
__device__ __forceinline__ void stream_init_barriers(uint64_t* full, int lane) {
    if (lane == 0) {
        for (int d = 0; d < kDepth; ++d) mbar_init(&full[d], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    __syncwarp();
}

}  // namespace psmc
