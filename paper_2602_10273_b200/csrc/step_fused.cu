// The whole per-token step as ONE kernel (16-byte aligned rows; groups of more than 32 particles get their update from
// a second, small kernel that follows this one: everything up to the rows' tokens and weights is done here): the loop body of
// Algorithm 1 without the cache move -- proposal sums (Corollary 1), token draw, Eq. 7, weight update, ESS (Eq. 5),
// trigger, resampling and slot map.
//
// How the logit block is dealt out.  Every row is cut into granules of 512 bytes; the R * granules-per-row granules
// of the block, in row-major order, are split into one contiguous share per CTA (one CTA per SM, shares differ by at
// most one granule).  A share meets a few rows: its "segments".  A segment that covers a whole row is LOCAL to the
// CTA; the first and the last segment of a share may be parts of rows shared with the neighbouring CTAs.  Each
// segment is split evenly among the CTA's streaming warps (a "piece" per warp, a few KB), which stream their pieces
// through private rings of bulk asynchronous copies exactly as the stand-alone logit pass does (logits_stream.cuh)
// and leave one (c, s1, sb) triple per piece: in shared memory for local segments, in global memory for shared rows.
// The shared parts are taken first, then the whole rows one after the other, so rows complete one after the other
// while the sweep is still running.
//
// Who finishes a row, and when.  Dependent trips to memory take several times longer while the sweep saturates HBM
// than after it, and a warp that polls takes issue slots from the warps that stream, so during the sweep only what
// must happen between CTAs happens, plus arithmetic on shared memory.  One extra warp per CTA, the helper, is parked
// on a named CTA barrier that the streaming warps of ITS OWN CTA arrive on (every wait is for warps that are resident
// by construction and whose own waits are bounded) until a segment is complete.  For the CTA's part of a shared row
// it then takes a ticket on the row's global counter: the CTA that draws the last ticket owns the row.  No CTA ever
// waits for another one.  For every row the CTA owns the helper forms the totals in fp64 from the triples (shared
// memory, or global memory for a shared row) and names the piece that holds U * sum; all of that hides behind the
// sweep except for the row streamed last.  After the sweep all warps of the CTA finish the rows it owns together, a
// team of up to eight warps per row: a re-read of the selected piece split over the team (a few KB, still in L2), the
// token, log p(y) and log omega (logits_common.cuh).  A finished row counts one arrival for its group, and the warp
// that brings a group to N arrivals runs the group's update (weights_core.cuh) on the spot.
//
// The finished flags are read from one array and written to another (they alternate from step to step): a group may
// close, and rewrite its flags, while other CTAs have not looked at the flags of their rows yet.  Arrival counters
// are put back to zero by the warp that draws the last ticket, on every path, so consecutive launches need no
// clearing.  The two counters of the move lists alternate between steps (the kernel clears the pair the next step
// will use), because a group may append to the lists while other CTAs are only starting.
#include <mutex>

#include "logits_stream.cuh"
#include "weights_core.cuh"

namespace psmc {
namespace {

constexpr int kGranule = 512;      // bytes: one 16-byte chunk per lane
constexpr int kStepWarps = 23;     // streaming warps per CTA at most (with the helper: 6 warps per scheduler, 80 registers)
constexpr int kMaxSegments = 48;   // rows one CTA's share may meet (shapes beyond that take the two-kernel step)
constexpr int kMinGranulesPerWarp = 8;  // 4 KB, one stage: on small blocks fewer, larger pieces mean fewer triples to sum per row (measured: 4 -> 8 saves 2.5 us per step on 16 x 151936 logits, 16 loses 0.7 again)
constexpr int kOneRowGranules = 256;  // rows up to this size (128 KB) go one to a CTA when the block has no more rows than SMs
constexpr int kStagedTriples = 256;  // triples of a shared row that are copied to shared memory before they are summed
static_assert(kStepWarps % 4 == 3, "the helper completes the last scheduler's set of warps");

// How a block is cut up; a pure function of (R, V, dtype), the same on host and device.
struct StepGeom {
    int gpr;          // granules per row
    int base, extra;  // a CTA's share: `base` granules, one more for the first `extra` CTAs
    int row_bytes16;  // bytes of a row that bulk copies can fetch (a multiple of 16)
    int tail;         // ragged logits after them
    int W;            // streaming warps per CTA
    int seg_cap;      // rows of the shared-memory triple table
    int per_row;      // CTAs per row when rows are dealt out one by one, else 0 (base / extra then count within a row)
};

struct StepParams {
    const void* logits;
    int R, V;
    int64_t ld;
    StepGeom g;
    FinishParams f;
    WeightsArgs a;
    float4* shared_triples;   // [grid][2][W]: triples of the parts of rows a CTA shares with its neighbours
    int32_t* row_arrivals;    // [R] CTAs that have delivered their part of a shared row
    int32_t* group_arrivals;  // [G] rows of the group that are finished
    int32_t* zero_words;
    int groups_here;          // 0: groups of more than 32 particles, updated by a kernel of their own after this one
};

// per_row == 0: the whole block is one run of granules dealt out evenly.  per_row = c > 0: every row is dealt to c
// CTAs of its own (CTA b holds part b % c of row b / c), so that no CTA meets two rows.
__host__ __device__ __forceinline__ int share_first(const StepGeom& g, int b) {
    if (g.per_row) {
        const int row = b / g.per_row, part = b - row * g.per_row;
        return row * g.gpr + part * g.base + (part < g.extra ? part : g.extra);
    }
    return b * g.base + (b < g.extra ? b : g.extra);
}
__host__ __device__ __forceinline__ int share_count(const StepGeom& g, int b) {
    const int place = g.per_row ? b % g.per_row : b;
    return g.base + (place < g.extra ? 1 : 0);
}
__host__ __device__ __forceinline__ int share_of(const StepGeom& g, int q) {  // the CTA whose share holds granule q
    const int big = g.extra * (g.base + 1);
    if (g.per_row) {
        const int row = q / g.gpr, r = q - row * g.gpr;
        return row * g.per_row + (r < big ? r / (g.base + 1) : g.extra + (r - big) / g.base);
    }
    return q < big ? q / (g.base + 1) : g.extra + (q - big) / g.base;
}

// One segment: the part of row `row` inside the share of CTA `b`.
struct Segment {
    int row;
    int g0, g1;  // granules [g0, g1) of the row
    int slot;    // which of the CTA's two global triple rows a shared part uses
    __device__ __forceinline__ bool local(const StepGeom& g) const { return g0 == 0 && g1 == g.gpr; }
};
// the part of row `row` inside the share [first, last) of granules
__device__ __forceinline__ Segment segment_in_share(const StepGeom& g, int first, int last, int row) {
    const int lo = max(first, row * g.gpr), hi = min(last, (row + 1) * g.gpr);
    Segment s;
    s.row = row;
    s.g0 = lo - row * g.gpr;
    s.g1 = hi - row * g.gpr;
    s.slot = (row == first / g.gpr) ? 0 : 1;
    return s;
}
__device__ __forceinline__ Segment segment_of_row(const StepGeom& g, int b, int row) {
    const int first = share_first(g, b);
    return segment_in_share(g, first, first + share_count(g, b), row);
}
// The CTA's segments in the order they are taken: the shared parts at the two ends first, then the rows in between.
__device__ __forceinline__ int segment_in_order(int k, int S) {
    if (S < 2) return 0;
    return k == 0 ? S - 1 : k - 1;
}
// A segment's granules are dealt to the W streaming warps in vocabulary order, warp 0 first, in proportion to the
// warps' weights.  A full CTA has 23 streaming warps and the helper: the scheduler that hosts the helper (warp 23,
// hence warps 3, 7, ... too) runs five streaming warps where the other three run six, the helper is parked on a
// barrier for nearly all of the sweep, and the sweep is close to what a scheduler can issue.  Measured on B200: with
// equal pieces those five warps end 3 us before the others, with 6/5 of a plain piece each 1 us after them, so they
// take 7/6.  Smaller CTAs deal evenly.
constexpr unsigned kFullWeight = 6 * kStepWarps + kStepWarps / 4;  // 18 warps of weight 6, 5 of weight 7
__device__ __forceinline__ unsigned weight_before(int place) { return 6u * (unsigned)place + (unsigned)place / 4u; }
__device__ __forceinline__ void piece_granules(const Segment& s, int place, int W, int& p0, int& p1) {
    const unsigned n = (unsigned)(s.g1 - s.g0);  // n * kFullWeight < 2^32, checked by the host
    if (W == kStepWarps) {  // division by a constant
        p0 = s.g0 + (int)(n * weight_before(place) / kFullWeight);
        p1 = s.g0 + (int)(n * weight_before(place + 1) / kFullWeight);
    } else {
        p0 = s.g0 + (int)(n * (unsigned)place / (unsigned)W);
        p1 = s.g0 + (int)(n * (unsigned)(place + 1) / (unsigned)W);
    }
}
// logits [a0, b0) of the row that a piece covers (the piece that holds a row's last granule also owns the ragged end)
template <int DT>
__device__ __forceinline__ void piece_logits(const StepGeom& g, int V, int p0, int p1, int& a0, int& b0) {
    constexpr int kPerGranule = kGranule / (DT == PSMC_F32 ? 4 : 2);
    a0 = p0 * kPerGranule;
    b0 = p1 == g.gpr ? V : p1 * kPerGranule;
    if (p1 <= p0) b0 = a0;
}

// One arrival on a global counter.  Release: what this thread wrote, and what it has observed of other threads' writes,
// is visible to whoever reads the new count; acquire: the writes of the earlier arrivals are visible to this thread
// (and, after a warp barrier, to its warp) once it holds the returned count.
__device__ __forceinline__ int arrive_acq_rel(int32_t* counter) {
    int old;
    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(counter) : "memory");
    return old;
}
// Named CTA barriers 1..15 as producer/consumer signals: the streaming warps arrive (and run on), the helper waits.
// The hardware parks the waiting warp, so it takes no issue slots while it waits and resumes with the last arrival.
constexpr int kNamedBarriers = 15;
__device__ __forceinline__ void named_arrive(int id, int threads) {
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void named_sync(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// Where a warp's k-th piece lies: pure geometry (a function of the launch parameters), so the first kPieceTab pieces
// of every warp are worked out before the kernel waits for its predecessor and kept in shared memory.  The index
// arithmetic (divisions by run-time values) would otherwise run at every piece boundary, in the producer as in the
// consumer, with the warp's ring running dry meanwhile.
constexpr int kPieceTab = 16;  // (6 cover the batched prompts; shares that meet 20-30 short rows: 3200 x 32000 bf16 77.3 -> 73.7 us)
struct PieceRec {
    long long off;   // first byte, relative to the start of the logit block
    int bytes;       // bytes bulk copies fetch (a multiple of 16)
    uint32_t meta;   // tail (bits 0-7) | segment (8-15) | local to the CTA (16) | slot of a shared part (17)
};

struct StepShared {
    uint64_t ring_bars[kStepWarps * kDepth];
    uint64_t seg_bars[kMaxSegments];       // one per segment: all streaming warps have stored their triple
    unsigned char seg_done[kMaxSegments];  // the segment's row is finished (absorbing EOS): nothing is read or summed
    double seg_u[kMaxSegments];            // the uniform of the segment's row (token stream of the counter hash)
    GroupScratch<32> sc;                   // the helper's; a streaming warp that closes a group uses its idle ring
    // rows this CTA finishes after the sweep, listed by the helper with their totals and the piece to re-read
    int n_pend, timed_out;
    int own_first, own_last;               // this CTA's share of granules (worked out once)
    PieceRec pieces[kStepWarps][kPieceTab];  // the first pieces of every streaming warp, laid out ahead of the sweep
    RowTotals pend_t[kMaxSegments];
    int pend_row[kMaxSegments], pend_a0[kMaxSegments], pend_b0[kMaxSegments];
    double end_tot[kStepWarps + 1];        // per warp: mass of its part of the selected piece
    float4 staged[kStagedTriples];         // the triples of a shared row, fetched in one go by the helper
};

// ---------------------------------------------------------------- streaming warps
struct PieceDesc {
    const char* src;   // first byte bulk copies fetch
    int bytes;         // how many (a multiple of 16)
    int tail;          // ragged logits after them, fetched with plain loads
    int seg, place;
    bool live;
    bool local;        // the piece's row lies wholly in this CTA's share
    int slot;          // else: which of the CTA's two global triple rows its part uses
};
// the geometry of piece k of warp `warp` in the share [own_first, own_last)
template <int DT>
__device__ __forceinline__ PieceRec piece_layout(const StepParams& sp, int own_first, int own_last, int first_row, int S,
                                                 int k, int warp) {
    constexpr int kEsize = DT == PSMC_F32 ? 4 : 2;
    const int seg = segment_in_order(k, S);
    const Segment s = segment_in_share(sp.g, own_first, own_last, first_row + seg);
    int p0, p1;
    piece_granules(s, warp, sp.g.W, p0, p1);
    PieceRec r;
    r.off = (long long)s.row * sp.ld * kEsize + (long long)p0 * kGranule;
    const int end = min(p1 * kGranule, sp.g.row_bytes16);
    r.bytes = max(end - p0 * kGranule, 0);
    const int tail = (p1 == sp.g.gpr && p1 > p0) ? sp.g.tail : 0;
    r.meta = (uint32_t)tail | ((uint32_t)seg << 8) | (s.local(sp.g) ? 1u << 16 : 0u) | ((uint32_t)s.slot << 17);
    return r;
}
template <int DT>
__device__ __forceinline__ PieceDesc piece_at(const StepParams& sp, const StepShared& sh, int first_row, int S, int k,
                                              int warp) {
    const PieceRec r = k < kPieceTab ? sh.pieces[warp][k]
                                     : piece_layout<DT>(sp, sh.own_first, sh.own_last, first_row, S, k, warp);
    PieceDesc d;
    d.src = reinterpret_cast<const char*>(sp.logits) + r.off;
    d.bytes = r.bytes;
    d.tail = (int)(r.meta & 255u);
    d.seg = (int)((r.meta >> 8) & 255u);
    d.place = warp;
    d.live = !sh.seg_done[d.seg];
    d.local = (r.meta >> 16) & 1u;
    d.slot = (int)((r.meta >> 17) & 1u);
    return d;
}

// The streaming loop of one warp over its pieces; the bulk-copy pipeline of logits_stream.cuh with one triple per
// piece.  Returns false when a bounded wait ran out (status raised, copies drained, every barrier still arrived on).
template <int DT, int MODE>
__device__ __forceinline__ bool stream_pieces(const StepParams& sp, StepShared& sh, float4* local_triples, int first_row,
                                              int S, int warp, int lane, unsigned char* ring, uint64_t* full) {
    const PackedConsts kc = packed_consts(sp.f.bf);
    const int W = sp.g.W;

    // The block is read once: its lines go into L2 marked evict-first, so that the sweep recycles its own lines instead
    // of pushing out what the kernel before left there (the dirty lines of a cache move would otherwise be written back
    // under this sweep: measured 48.8 -> 46.1 us per step inside the decoding loop, and 2 us per step less overall).
    // The segment streamed last keeps the normal priority: one piece of it is read again when the row is finished.
    const uint64_t policy = l2_policy_evict_first();
    const int hint_until = S - 1;
    // producer cursor (the same in every lane; lane 0 issues)
    int pk = 0, p_left = 0;
    const char* p_src = nullptr;
    auto prod_seek = [&]() {
        for (; pk < S; ++pk) {
            const PieceDesc d = piece_at<DT>(sp, sh, first_row, S, pk, warp);
            if (d.live && d.bytes > 0) {
                p_src = d.src;
                p_left = d.bytes;
                return;
            }
        }
    };
    int issued = 0;
    auto issue = [&]() {
        if (p_left == 0) return;
        const int bytes = p_left < kStageBytes ? p_left : kStageBytes;
        if (lane == 0) {
            const int slot = issued & (kDepth - 1);
            fence_async_smem();  // the stage's previous contents were read through the generic proxy
            mbar_expect_tx(&full[slot], (uint32_t)bytes);
            if (pk < hint_until) bulk_load_hint(ring + (size_t)slot * kStageBytes, p_src, (uint32_t)bytes, &full[slot], policy);
            else bulk_load(ring + (size_t)slot * kStageBytes, p_src, (uint32_t)bytes, &full[slot]);
        }
        ++issued;
        p_src += bytes;
        p_left -= bytes;
        if (p_left == 0) {
            ++pk;
            prod_seek();
        }
    };
    static_assert((kDepth & (kDepth - 1)) == 0, "the ring depth is a power of two");

    prod_seek();
    for (int d = 0; d < kDepth - 1; ++d) issue();

    bool failed = false;
    int consumed = 0;
    for (int ck = 0; ck < S; ++ck) {
        const PieceDesc d = piece_at<DT>(sp, sh, first_row, S, ck, warp);
        if (!d.live) continue;  // finished row: no triple, no arrival (the finisher does not wait for it either)
        LaneSums acc = lane_sums_init();
        __nv_bfloat162 thr2 = __float2bfloat162_rn(acc.thr);
        int left = failed ? 0 : d.bytes;
        while (left > 0) {
            __syncwarp();  // every lane is done with the stage that is about to be refilled
            issue();
            const int slot = consumed & (kDepth - 1);
            if (!__all_sync(kFull, mbar_wait(&full[slot], (uint32_t)((consumed / kDepth) & 1)))) {  // the same answer in every lane
                failed = true;
                break;
            }
            const uint4* st = reinterpret_cast<const uint4*>(ring + (size_t)slot * kStageBytes);
            const int bytes = left < kStageBytes ? left : kStageBytes;
            const int chunks = bytes >> 4;
            int c0 = 0;
            for (; c0 + 128 <= chunks; c0 += 128) {  // 2 KB = four 16-byte chunks per lane at a time
                const uint4 v0 = st[c0 + lane], v1 = st[c0 + 32 + lane], v2 = st[c0 + 64 + lane], v3 = st[c0 + 96 + lane];
                const uint32_t w[16] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w,
                                        v2.x, v2.y, v2.z, v2.w, v3.x, v3.y, v3.z, v3.w};
                consume<DT, MODE, 16>(w, kc, acc, thr2);
            }
            constexpr uint32_t kNoLogit = DT == PSMC_BF16 ? 0xff80ff80u : 0xff800000u;  // -inf: no mass, never a maximum
            for (; c0 < chunks; c0 += 32) {  // the same trip count in every lane
                const bool in = c0 + lane < chunks;
                const uint4 v0 = in ? st[c0 + lane] : make_uint4(kNoLogit, kNoLogit, kNoLogit, kNoLogit);
                const uint32_t w[4] = {v0.x, v0.y, v0.z, v0.w};
                consume<DT, MODE, 4>(w, kc, acc, thr2);
            }
            ++consumed;
            left -= bytes;
        }
        if (failed) {  // a triple without mass: the row gets flagged, the barrier still gets its arrival
            acc = lane_sums_init();
            if (lane == 0) sh.timed_out = 1;
        } else if (d.tail > 0) {  // ragged end of the row
            add_one<MODE>(lane < d.tail ? load_elem<DT>(d.src + d.bytes, lane) : -INFINITY, kc, acc);
        }
        const float s1 = warp_sum(pair_sum(add2(acc.s1a, acc.s1b)));
        const float sb = (MODE == kBeta1) ? 0.f : warp_sum(pair_sum(add2(acc.sba, acc.sbb)));
        if (lane == 0) {
            const float4 tr = make_float4(-acc.neg_c, s1, sb, 0.f);
            if (d.local) local_triples[d.seg * W + d.place] = tr;
            else __stcg(&sp.shared_triples[((size_t)blockIdx.x * 2 + d.slot) * W + d.place], tr);
            // release: the triple is visible to whoever sees the barrier complete
            if (S > kNamedBarriers) mbar_arrive(&sh.seg_bars[d.seg]);
        }
        if (S <= kNamedBarriers) named_arrive(1 + ck, (W + 1) * 32);  // the triple is stored: tell the helper, do not wait
    }
    if (failed) {
        if (lane == 0) raise_status(sp.a.status, PSMC_E_TIMEOUT);
        // do not leave with copies still landing in this CTA's shared memory: bounded second wait
        for (int j = consumed; j < issued; ++j) mbar_wait(&full[j & (kDepth - 1)], (uint32_t)((j / kDepth) & 1));
    }
    return !failed;
}

// ---------------------------------------------------------------- finishing a row
// Row totals from the triples of a local row (shared memory, W of them) or of a shared row (global memory, W from each
// CTA that holds a part, in CTA order = vocabulary order).  Every lane gets the same result.
template <int MODE>
__device__ __forceinline__ RowTotals row_totals(const StepParams& sp, StepShared& sh, const float4* local_triples,
                                                const Segment& s, int seg, int c_first, int c_last, double U, int lane) {
    const int W = sp.g.W;
    if (s.local(sp.g)) {  // at most kStepWarps <= 32 triples: one per lane
        const float4 f = lane < W ? local_triples[seg * W + lane] : make_float4(kRefFloor, 0.f, 0.f, 0.f);
        return combine_triples_32<MODE>(f, sp.f.beta, U, lane);
    }
    const int row = s.row, n = (c_last - c_first + 1) * W;
    auto from_global = [&](int j) {
        const int c = c_first + j / W, place = j - (j / W) * W;
        const int slot = (row == share_first(sp.g, c) / sp.g.gpr) ? 0 : 1;
        return __ldcg(&sp.shared_triples[((size_t)c * 2 + slot) * W + place]);
    };
    if (n <= kStagedTriples) {
        // One trip to L2 for all of them (independent loads, issued back to back) instead of one per sweep of the
        // combination: on small blocks this is on the path that every step waits for.
        for (int j = lane; j < n; j += 32) sh.staged[j] = from_global(j);
        __syncwarp();
        return combine_triples<MODE>([&](int j) { return sh.staged[j]; }, n, sp.f.beta, U, lane);
    }
    return combine_triples<MODE>(from_global, n, sp.f.beta, U, lane);
}
// the logits the selected triple stands for
template <int DT>
__device__ __forceinline__ void selected_range(const StepParams& sp, const Segment& s, int c_first, int jsel, int& a0, int& b0) {
    const int W = sp.g.W;
    Segment part = s;
    int place = jsel;
    if (!s.local(sp.g)) {
        part = segment_of_row(sp.g, c_first + jsel / W, s.row);
        place = jsel % W;
    }
    int p0, p1;
    piece_granules(part, place, W, p0, p1);
    piece_logits<DT>(sp.g, sp.V, p0, p1, a0, b0);
}

// A row's result goes to memory and its group gets one arrival; the warp that completes the group updates it.
// Called by all 32 lanes of one warp.  rr == nullptr: the row is finished (absorbing EOS) and has nothing to store.
__device__ __forceinline__ void row_arrives(const StepParams& sp, StepShared& sh, GroupScratch<32>& sc, int row,
                                            const RowResult* rr, bool timed_out, int lane) {
    const WeightsArgs& a = sp.a;
    const int N = a.N, g = row / N;
    if (rr && lane == 0) {
        if (timed_out) raise_status(a.status, PSMC_E_TIMEOUT);
        else if (rr->tok < 0) raise_status(a.status, PSMC_E_NUMERIC);
        a.tok[row] = rr->tok;
        a.logp[row] = rr->logp;
        a.loginc[row] = rr->loginc;
    }
    if (!sp.groups_here) return;  // the rows' results are in memory: all this kernel owes a large group
    // The group's state as the step found it (nobody writes it before the group is complete) is asked for now: should
    // this warp turn out to be the one that completes the group, the loads have overlapped the trip of the ticket.
    ParticleState st{};
    if (lane < N) st = load_particle(a, g * N + lane);
    int ticket = 0;
    if (lane == 0) ticket = arrive_acq_rel(&sp.group_arrivals[g]);  // the row's result first, then the arrival
    ticket = __shfl_sync(kFull, ticket, 0);
    if (ticket != N - 1) return;
    // the group is complete: this warp updates it
    if (lane == 0) sp.group_arrivals[g] = 0;
    __syncwarp();
    int tk = -1;
    double lp = 0.0, inc = 0.0;
    if (lane < N) {  // one trip to memory for the rows' results (what a finished row has there is not used)
        const int r = g * N + lane;
        tk = __ldcg(const_cast<const int32_t*>(a.tok) + r);
        lp = __ldcg(const_cast<const double*>(a.logp) + r);
        inc = __ldcg(const_cast<const double*>(a.loginc) + r);
    }
    group_update(a, g, lane, 1, sc, tk, lp, inc, st);
    __syncwarp();  // sc is reused by the next group this warp closes
}

// The helper warp, during the sweep: lists the rows this CTA will finish, each with its totals (fp64, from the
// triples) and the piece that holds the target.  It follows the segments in the order they are streamed and waits for
// each on the segment's mbarrier, so all of this hides behind the sweep except for the segment streamed last.  For the
// CTA's part of a shared row it takes the CTA's ticket first and goes on only with the last ticket.  A finished row
// (absorbing EOS) is reported to its group by the CTA that holds the row's last granule.
template <int DT, int MODE>
__device__ __noinline__ void helper_warp(const StepParams& sp, StepShared& sh, const float4* local_triples, int first_row,
                                         int S, int lane) {
    const WeightsArgs& a = sp.a;
    const int N = a.N;
    for (int seg = lane; seg < S; seg += 32) {  // everything that does not depend on the sweep, ahead of it
        const int row = first_row + seg, g = row / N;
        sh.seg_u[seg] = hash_uniform(hash5(a.seed, kStreamToken, (uint64_t)g, (uint64_t)a.t, (uint64_t)(row - g * N)));
    }
    __syncwarp();
    for (int k = 0; k < S; ++k) {
        const int seg = segment_in_order(k, S);
        const Segment s = segment_in_share(sp.g, sh.own_first, sh.own_last, first_row + seg);
        const int row = s.row;
        if (sh.seg_done[seg]) {
            if (s.g1 == sp.g.gpr) row_arrives(sp, sh, sh.sc, row, nullptr, false, lane);
            continue;
        }
        int c_first = (int)blockIdx.x, c_last = (int)blockIdx.x;
        if (!s.local(sp.g)) {
            c_first = share_of(sp.g, row * sp.g.gpr);
            c_last = share_of(sp.g, (row + 1) * sp.g.gpr - 1);
        }
        // Every streaming warp of this CTA has stored its triple of the segment.  Each of them gets there in bounded
        // time (its own waits are bounded and it arrives whatever happens), so this wait ends.
        if (S <= kNamedBarriers) named_sync(1 + k, (sp.g.W + 1) * 32);
        int mine = 1;
        if (lane == 0) {
            if (S > kNamedBarriers && !mbar_wait_idle(&sh.seg_bars[seg], 0)) sh.timed_out = 1;
            if (c_last > c_first) {  // this CTA's triples first, then its ticket
                mine = arrive_acq_rel(&sp.row_arrivals[row]) == c_last - c_first ? 1 : 0;
                if (mine) sp.row_arrivals[row] = 0;  // every part has arrived: ready for the next launch
            }
        }
        mine = __shfl_sync(kFull, mine, 0);
        if (!mine) continue;
        RowTotals t = row_totals<MODE>(sp, sh, local_triples, s, seg, c_first, c_last, sh.seg_u[seg], lane);
        int a0 = 0, b0 = 0;
        if (t.ok) selected_range<DT>(sp, s, c_first, t.jsel, a0, b0);
        if (lane == 0) {
            // The piece that holds the target is read again when the row is finished, after the sweep.  Its lines were
            // fetched marked evict-first and are gone from L2 by then (the block is larger than L2); asked for again
            // now, they wait in L2 with the normal priority and the re-read costs a trip to L2 instead of one to HBM.
            constexpr int kEs = DT == PSMC_F32 ? 4 : 2;
            const int64_t from = (int64_t)a0 * kEs;
            const int bytes = (int)((((int64_t)b0 * kEs) & ~(int64_t)15) - from);  // (a piece starts on a granule)
            if (t.ok && k < S - 1 && bytes > 0)
                bulk_prefetch_l2(reinterpret_cast<const char*>(sp.logits) + (size_t)row * sp.ld * kEs + from, (uint32_t)bytes);
            const int i = sh.n_pend++;
            sh.pend_t[i] = t;
            sh.pend_row[i] = row;
            sh.pend_a0[i] = a0;
            sh.pend_b0[i] = b0;
        }
        __syncwarp();
    }
}

// After the sweep, every thread of the CTA: the pending rows, (warps / wpr) at a time.  The wpr warps of a row's team
// share the re-read of the piece that holds the target (contiguous 16-byte chunks per thread); the warp whose threads
// reach the target names the token and reports the row.  (A team need not be a power of two of warps.)
template <int DT, int MODE>
__device__ __noinline__ void finish_pending(const StepParams& sp, StepShared& sh, unsigned char* rings) {
    constexpr int kPer = DT == PSMC_BF16 ? 8 : 4;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const int n = sh.n_pend;
    const bool timed_out = sh.timed_out != 0;
    const int wpr = max(1, min(8, n_warps / n));  // warps per row: all of the CTA's warps shared out, eight at most
    const int rows_per_pass = n_warps / wpr;
    const int kk = warp / wpr, q = warp - kk * wpr;
    // a streaming warp's ring is idle by now: room for the group update's scratch
    GroupScratch<32>& sc = warp < sp.g.W ? *reinterpret_cast<GroupScratch<32>*>(rings + (size_t)warp * kDepth * kStageBytes)
                                         : sh.sc;
    for (int k0 = 0; k0 < n; k0 += rows_per_pass) {
        // ---- wpr warps per row: mass of each part of the selected piece ----
        const bool active = kk < rows_per_pass && k0 + kk < n;
        RowTotals t;
        t.ok = false;
        int row = 0, a0 = 0, b0 = 0, E = 0;
        const void* rowp = nullptr;
        float neg_C = 0.f;
        double lm = 0.0, incl = 0.0;
        if (active) {
            t = sh.pend_t[k0 + kk];
            if (timed_out) t.ok = false;
            row = sh.pend_row[k0 + kk];
            rowp = reinterpret_cast<const char*>(sp.logits) + (size_t)row * sp.ld * (DT == PSMC_F32 ? 4 : 2);
            if (t.ok) {
                a0 = sh.pend_a0[k0 + kk];
                b0 = sh.pend_b0[k0 + kk];
                neg_C = -t.C;
                const int chunks = (b0 - a0 + kPer - 1) / kPer, team = wpr * 32;
                E = ((chunks + team - 1) / team) * kPer;  // logits per thread
                lm = lane_share<DT, MODE, 8>(sp.f, rowp, a0 + (q * 32 + lane) * E, E, b0, neg_C);
                incl = warp_scan_incl(lm, lane);
            }
            if (lane == 31) sh.end_tot[warp] = incl;
        }
        __syncthreads();
        // ---- the warp whose threads reach the target: the token ----
        if (active) {
            const int w0 = warp - q;  // first warp of this row's team
            if (!t.ok) {
                if (q == 0) {
                    const RowResult bad{-1, 0.0, 0.0};
                    row_arrives(sp, sh, sc, row, &bad, timed_out, lane);
                }
            } else {
                // which part of the piece reaches the target: the same additions, in the same order, in every warp
                double cum = t.base, before = t.base;
                int first_hit = -1;
                for (int i = 0; i < wpr; ++i) {
                    if (i == q) before = cum;
                    const double ti = sh.end_tot[w0 + i];
                    cum += ti;
                    if (first_hit < 0 && ti > 0.0 && cum >= t.target) first_hit = i;
                }
                int y = -1;
                bool mine = false;
                if (first_hit == q) {
                    mine = true;
                    const double r_incl = before + incl;
                    const unsigned hit = __ballot_sync(kFull, lm > 0.0 && r_incl >= t.target);
                    const int owner = hit ? __ffs(hit) - 1 : 31;
                    const double run = __shfl_sync(kFull, r_incl - lm, owner);
                    const int o0 = a0 + (q * 32 + owner) * E;
                    y = locate_in_lane<DT, MODE>(sp.f, rowp, o0, min(b0, o0 + E), run, t.target, neg_C, lane);
                } else if (first_hit < 0 && q == 0) {
                    mine = true;  // the re-read sums fall short of the target: last token with mass in the piece
                    y = last_with_mass<DT, MODE>(sp.f, rowp, a0, b0, neg_C, lane);
                }
                if (mine) {
                    RowResult rr{-1, 0.0, 0.0};
                    if (y >= 0) rr = row_result<DT, MODE>(sp.f, rowp, t, y, lane);
                    row_arrives(sp, sh, sc, row, &rr, false, lane);
                }
            }
        }
        if (k0 + rows_per_pass < n) __syncthreads();  // sh.end_tot is reused by the next pass
    }
}

template <int DT, int MODE>
__global__ void __launch_bounds__((kStepWarps + 1) * 32, 1) psmc_step_kernel(const __grid_constant__ StepParams sp) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ StepShared sh;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int W = sp.g.W;
    float4* local_triples = reinterpret_cast<float4*>(smem + (size_t)W * kDepth * kStageBytes);
    const int first = share_first(sp.g, (int)blockIdx.x), count = share_count(sp.g, (int)blockIdx.x);
    const int first_row = first / sp.g.gpr;
    const int S = (first + count - 1) / sp.g.gpr - first_row + 1;  // <= sp.g.seg_cap, checked by the host

    if (warp < W) stream_init_barriers(sh.ring_bars + warp * kDepth, lane);
    if ((int)threadIdx.x < S) mbar_init(&sh.seg_bars[threadIdx.x], (uint32_t)W);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (warp < W && lane < kPieceTab && lane < S)  // one lane per piece; read back only by this warp
        sh.pieces[warp][lane] = piece_layout<DT>(sp, first, first + count, first_row, S, lane, warp);
    __syncwarp();
    chain_begin();  // everything above is local set-up; global memory from here on
    if (sp.zero_words && blockIdx.x == 0 && threadIdx.x < 2) sp.zero_words[threadIdx.x] = 0;
    if ((int)threadIdx.x < S) sh.seg_done[threadIdx.x] = sp.a.done[first_row + threadIdx.x];
    if (threadIdx.x == 0) {
        sh.n_pend = sh.timed_out = 0;
        sh.own_first = first;
        sh.own_last = first + count;
    }
    __syncthreads();

    if (warp < W) {
        stream_pieces<DT, MODE>(sp, sh, local_triples, first_row, S, warp, lane, smem + (size_t)warp * kDepth * kStageBytes,
                                sh.ring_bars + warp * kDepth);
    } else {
        helper_warp<DT, MODE>(sp, sh, local_triples, first_row, S, lane);
    }
    __syncthreads();  // the sweep is over, every bulk copy has landed and been summed; sh lists this CTA's rows
    if (sh.n_pend > 0) finish_pending<DT, MODE>(sp, sh, smem);
}

typedef void (*StepFn)(const StepParams);
template <int DT>
StepFn pick_step(int mode) {
    switch (mode) {
        case kBeta1: return psmc_step_kernel<DT, kBeta1>;
        case kBeta2: return psmc_step_kernel<DT, kBeta2>;
        case kBeta4: return psmc_step_kernel<DT, kBeta4>;
        case kBeta8: return psmc_step_kernel<DT, kBeta8>;
        default: return psmc_step_kernel<DT, kBetaAny>;
    }
}

// false: the shape does not fit the one-kernel step
bool step_geometry(int R, int V, int dt, StepGeom& g, int& grid) {
    const int esize = dt == PSMC_F32 ? 4 : 2, per16 = 16 / esize;
    const int64_t row_bytes16 = (int64_t)(V / per16) * 16;
    const int64_t gpr = row_bytes16 > 0 ? (row_bytes16 + kGranule - 1) / kGranule : 1;
    const int64_t total = (int64_t)R * gpr;
    if (total >= (int64_t)1 << 30 || gpr * 256 >= (int64_t)1 << 32) return false;
    grid = (int)(total < kSMs ? total : kSMs);
    g.gpr = (int)gpr;
    g.base = (int)(total / grid);
    g.extra = (int)(total % grid);
    // A small block is all latency: with one whole row per CTA no row is shared between CTAs, which takes the row
    // ticket and the trip for the other CTAs' triples out of the chain every step waits for.  Measured (launches back
    // to back): 4 x 1024 fp32 12.4 -> 10.6 us, 8 x 32000 bf16 14.9 -> 12.2 us; rows of 300 KB lose (16 x 151936 bf16:
    // 18.6 -> 21.0 us, one SM streams a row in 3 us), so the rule stops at 128 KB.
    g.per_row = 0;
    if (R <= kSMs && gpr <= kOneRowGranules) {
        grid = R;
        g.base = (int)gpr;
        g.extra = 0;
    }
    // Larger rows of a block with no more rows than SMs: c = SMs / R CTAs per row (one whole row per CTA from 75 rows
    // on), so that every CTA streams one part of one row (one ticket, no tiny pieces at a boundary between two rows;
    // with c = 1 no ticket at all).  Measured along a run with resampling, rows of 151936 bf16 logits: 16 rows
    // 20.7 -> 20.3 us per step, 32 rows 24.0 -> 23.0 us, 64 rows 28.2 -> 23.6 us, 100 rows 31.2 -> 23.3 us, 128 rows
    // 33.4 -> 23.7 us.  (Whole rows for larger blocks, three or four to a CTA, lose more to the uneven shares than
    // they gain: 512 x 128256 37.9 -> 39.7 us.)
    else if (R <= kSMs && gpr >= 2 * (kSMs / R)) {
        g.per_row = kSMs / R;
        grid = R * g.per_row;
        g.base = (int)(gpr / g.per_row);
        g.extra = (int)(gpr % g.per_row);
    }
    g.row_bytes16 = (int)row_bytes16;
    g.tail = V % per16;
    const int per_cta = g.base + (g.extra ? 1 : 0);
    int W = (per_cta + kMinGranulesPerWarp - 1) / kMinGranulesPerWarp;
    g.W = W < 1 ? 1 : (W > kStepWarps ? kStepWarps : W);
    g.seg_cap = (int)((per_cta + gpr - 2) / gpr + 1);
    return g.seg_cap <= kMaxSegments;
}

}  // namespace

size_t step_fused_scratch_bytes() { return (size_t)kSMs * 2 * kStepWarps * sizeof(float4); }

// This kernel needs rows that bulk copies can fetch (16-byte aligned starts) and a share per CTA that meets at most
// kMaxSegments rows; everything else takes the step as two kernels (logits_pass.cu, weights_resample.cu).  A group
// that one warp can update (N <= 32) is updated here by the warp that finishes its last row; larger groups by
// rows_weights_kernel right after (measured with 151936 bf16 logits per row, launches back to back: 64 particles
// 41.4 -> 23.6 us per step, 128 particles 73.9 -> 23.7 us against the step as two kernels).
bool step_can_fuse(const LogitsStreamArgs& la, int N) {
    const LogitsGeometry lg = logits_geometry(la.logits, la.dt, la.R, la.V, la.ld, la.beta);
    StepGeom g;
    int grid;
    (void)N;  // groups of more than 32 particles take the sweep and the rows from this kernel, the update from another
    return lg.vec != 0 && step_geometry(la.R, la.V, la.dt, g, grid);
}

cudaError_t launch_step_fused(const LogitsStreamArgs& la, const WeightsArgs& wa, void* shared_triples,
                              int32_t* row_arrivals, int32_t* group_arrivals, cudaStream_t stream) {
    const LogitsGeometry lg = logits_geometry(la.logits, la.dt, la.R, la.V, la.ld, la.beta);
    StepParams sp;
    int grid;
    if (!step_geometry(la.R, la.V, la.dt, sp.g, grid)) return cudaErrorInvalidValue;
    sp.logits = la.logits; sp.R = la.R; sp.V = la.V; sp.ld = la.ld;
    sp.f.logits = la.logits; sp.f.V = la.V; sp.f.ld = la.ld; sp.f.span = 0; sp.f.n_spans = 0; sp.f.partials = nullptr;
    sp.f.beta = wa.beta; sp.f.alpha_t = wa.alpha_t; sp.f.bf = lg.bf; sp.f.vec = lg.vec;
    sp.a = wa;
    sp.shared_triples = reinterpret_cast<float4*>(shared_triples);
    sp.row_arrivals = row_arrivals;
    sp.group_arrivals = group_arrivals;
    sp.zero_words = la.zero_words;
    sp.groups_here = wa.N <= 32 ? 1 : 0;
    const size_t smem = (size_t)sp.g.W * kDepth * kStageBytes + (size_t)sp.g.seg_cap * sp.g.W * sizeof(float4);
    StepFn fn = la.dt == PSMC_F32 ? pick_step<PSMC_F32>(lg.mode) : pick_step<PSMC_BF16>(lg.mode);
    cudaError_t e = allow_dynamic_smem(reinterpret_cast<const void*>(fn),
                                       kStepWarps * kDepth * kStageBytes + kMaxSegments * kStepWarps * (int)sizeof(float4));
    if (e != cudaSuccess) return e;
    e = launch_chained(fn, dim3((unsigned)grid), dim3((unsigned)((sp.g.W + 1) * 32)), smem, stream, sp);
    if (e != cudaSuccess || sp.groups_here) return e;
    return launch_rows_weights(wa, stream);
}

}  // namespace psmc

// ---- host-only queries of the dealing (tests of the geometry need no GPU) ----
extern "C" psmc_status psmc_step_layout(int R, int V, psmc_dtype dt, int32_t* layout_out, int32_t* shares_out,
                                        int shares_cap) {
    if (R <= 0 || V <= 0 || (dt != PSMC_F32 && dt != PSMC_BF16) || !layout_out) return PSMC_E_INVAL;
    psmc::StepGeom g;
    int grid = 0;
    const bool ok = psmc::step_geometry(R, V, dt, g, grid);
    layout_out[0] = ok ? 1 : 0;
    layout_out[1] = grid;
    layout_out[2] = g.W;
    layout_out[3] = g.gpr;
    layout_out[4] = g.seg_cap;
    layout_out[5] = g.per_row;
    layout_out[6] = g.row_bytes16;
    layout_out[7] = g.tail;
    if (shares_out) {
        if (shares_cap < grid + 1) return PSMC_E_INVAL;
        for (int b = 0; b < grid; ++b) shares_out[b] = psmc::share_first(g, b);
        shares_out[grid] = psmc::share_first(g, grid - 1) + psmc::share_count(g, grid - 1);
    }
    return PSMC_OK;
}
extern "C" int psmc_step_share_of(int R, int V, psmc_dtype dt, int granule) {
    psmc::StepGeom g;
    int grid = 0;
    if (R <= 0 || V <= 0 || (dt != PSMC_F32 && dt != PSMC_BF16) || !psmc::step_geometry(R, V, dt, g, grid)) return -1;
    if (granule < 0 || (int64_t)granule >= (int64_t)R * g.gpr) return -1;
    return psmc::share_of(g, granule);
}

