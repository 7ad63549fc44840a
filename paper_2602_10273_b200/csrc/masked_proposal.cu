// The logit pass with the proposal restricted to a set S of tokens: the top_k tokens of the row by logit, or the
// nucleus holding a share top_p of the tempered distribution softmax(beta l).  Tokens rank by logit, lower id first
// among equal logits; S is the first k of that ranking.  Eq. 7 takes the proposal actually sampled from,
//   q_S(v) = exp(beta l_v) / sum_{u in S} exp(beta l_u) on S,   log omega = alpha_t log p(y) - log q_S(y),
// with p the softmax over the WHOLE row.
//
// One CTA per row.  A logit's bit pattern maps to an unsigned key that orders like the value, so S is
// {key > T} plus the first `need` tokens with key == T in id order.
//
// A top_k of up to half the number of shares goes by a threshold: every thread sees its own share of the row, cut
// once more into 8 (bf16) or 4 (fp32) sub-shares by position inside the 16-byte vectors -- 4096 or 2048 shares for 512
// threads -- so the k-th largest of the shares' maxima has at least k logits at or above it (and, the shares being
// interleaved, not many more).  One sweep finds the maxima, a second collects the logits at or above the threshold into a candidate list in
// shared memory (and sums the normaliser of p), and the search for (T, need) runs on that list.
//
// A nucleus of share top_p <= 0.9999 goes by a floor on the mass: tokens lighter than (1 - top_p) / V of the row's mass
// cannot belong to it (all of them together weigh less than 1 - top_p).  Three sweeps: the largest logit; the row's
// masses under p and under the proposal; the tokens above the floor into the list.
//
// Otherwise (T, need) come from a radix search over the key, 8 bits a level from the top (2 levels for bf16, 4 for
// fp32): a level counts, per digit, the tokens whose higher digits equal the prefix found so far -- and for the
// nucleus their mass 2^{beta (x - C)} as a 64-bit fixed-point number (2^-40 units, integer adds: the totals do not
// depend on the order of the atomics) -- then picks the digit in which the running count reaches k (the running mass
// reaches top_p of the total).  Counters live in shared memory as [digit][lane] columns (masses: two lanes a column),
// so the lanes of a warp do not pile up on an address however the logits cluster.  Tokens with equal key have equal
// mass, so on the last level need = ceil(remaining mass / mass of one).  Sweeps over the row when counting:
//   1  the largest logit, NaN / +inf check; for top-k also the counts of the first level (digits need no reference)
//   2  nucleus only: counts and masses of the first level
//   3  the second level, and sum 2^{x - C} over the whole row (the normaliser of p)
//   4  every token whose leading 16 key bits are at or above the 16 chosen goes to the candidate list (id, bits): for
//      bf16 exactly S and the ties at the cut, for fp32 also the tokens that agree with the cut to bf16 precision
//
// Everything else works on the list: the levels not yet decided; then the candidates at or above the cut are kept and
// sorted by id (bitonic; k plus the ties at the cut, a short list), and the ties' ranks, the masses of S and the
// inverse CDF are block scans over threads that hold consecutive entries.  The first sweep comes from HBM, the others
// mostly from L2; all use 16-byte loads, four in flight per thread.  Rows whose candidates do not fit the list (a
// top_k in the tens of thousands, a nearly flat nucleus, a crowd of equal logits) fall back to sweeps over the row
// for every remaining step.
#include "internal.h"
#include "logits_common.cuh"
#include "logits_stream.cuh"
#include "weights_core.cuh"

namespace psmc {
namespace {

constexpr int kDigits = 256;
constexpr float kFixOne = 1099511627776.f;  // 2^40: fixed-point unit of the nucleus masses (masses are <= 1)
// Dynamic shared memory: the counters ([256][32] counts; for the nucleus also [256][16] 64-bit masses, two lanes a
// column), then the candidate list (8 bytes an entry).  The counters' memory later takes the sorted list, so the
// list is no longer than the counts are.  64 KB (top-k) or 96 KB (nucleus) in all, so two CTAs of 512 threads share
// an SM: one sweeps its row while the other is in the barrier-heavy work on its list.
constexpr int kCountBytes = kDigits * 32 * 4, kMassBytes = kDigits * 16 * 8;
constexpr int kListCap = kCountBytes / 8;  // 4096 entries

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
    constexpr int kTop = DT == PSMC_BF16 ? 15 : 31;
    constexpr uint32_t sign = 1u << kTop, all = DT == PSMC_BF16 ? 0xffffu : 0xffffffffu;
    // negative values: every bit flipped; others: the sign bit set.  -0 would land one below +0: moved up onto it.
    const uint32_t key = (b ^ ((0u - (b >> kTop)) | sign)) & all;
    return key + (key == sign - 1u);
}
// the bit pattern a key came from (of +0 for the key the two zeros share)
template <int DT>
__device__ __forceinline__ uint32_t bits_of_key(uint32_t key) {
    constexpr int kTop = DT == PSMC_BF16 ? 15 : 31;
    constexpr uint32_t sign = 1u << kTop, all = DT == PSMC_BF16 ? 0xffffu : 0xffffffffu;
    return (key & sign) ? (key ^ sign) : (~key & all);
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

// Two bf16 logits in one word, handled by the packed bf16 instructions.  The maximum is the NaN-propagating one (a
// NaN of either sign anywhere in a share makes the share's maximum a NaN, whose key ranks above +inf's); +0 and -0
// compare equal, as their keys do.
__device__ __forceinline__ __nv_bfloat162 as_bf162(uint32_t w) {
    __nv_bfloat162 r;
    *reinterpret_cast<uint32_t*>(&r) = w;
    return r;
}
__device__ __forceinline__ uint32_t max_nan_pair(uint32_t a, uint32_t b) {
    const __nv_bfloat162 m = __hmax2_nan(as_bf162(a), as_bf162(b));
    return *reinterpret_cast<const uint32_t*>(&m);
}
// 0xffff in each half of the word whose logit is >= the threshold's (no NaN on either side)
__device__ __forceinline__ uint32_t ge_pair(uint32_t w, uint32_t th2) { return __hge2_mask(as_bf162(w), as_bf162(th2)); }
// the bf16 pattern (in both halves of a word) that compares like `key`: every logit with a key >= key is >= it
__device__ __forceinline__ uint32_t pair_threshold(uint32_t key) {
    constexpr uint32_t kNegInfKey = 0x007fu;
    const uint32_t k = key < kNegInfKey ? kNegInfKey : key;  // below -inf's key: everything passes
    const uint32_t sign = 0x8000u;
    const uint32_t b = (k & sign) ? (k ^ sign) : (~k & 0xffffu);
    return b | (b << 16);
}

// The row in no particular order: fv(v, id of its first logit) for every aligned 16 bytes between the first and the
// last 16-byte boundary (four loads in flight per thread), fs(bits, id) for the logits of the ragged ends.
template <int DT, class FV, class FS>
__device__ __forceinline__ void for_each_vector(const void* rowp, int V, FV fv, FS fs) {
    constexpr int kPer = DT == PSMC_BF16 ? 8 : 4, kEs = DT == PSMC_BF16 ? 2 : 4;
    int head = (int)(((16 - (reinterpret_cast<uintptr_t>(rowp) & 15)) & 15) / kEs);
    if (head > V) head = V;
    const int nvec = (V - head) / kPer, tail0 = head + nvec * kPer;
    const uint4* q = reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(rowp) + (size_t)head * kEs);
    const int stride = (int)blockDim.x;
    int j0 = (int)threadIdx.x;
    for (; j0 + 3 * stride < nvec; j0 += 4 * stride) {  // full rounds: no bounds checks between the loads
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = __ldg(&q[j0 + u * stride]);
#pragma unroll
        for (int u = 0; u < 4; ++u) fv(v[u], head + (j0 + u * stride) * kPer);
    }
    for (; j0 < nvec; j0 += stride) fv(__ldg(&q[j0]), head + j0 * kPer);
    for (int i = threadIdx.x; i < head; i += blockDim.x) fs(load_bits<DT>(rowp, i), i);
    for (int i = tail0 + threadIdx.x; i < V; i += blockDim.x) fs(load_bits<DT>(rowp, i), i);
}

// f(bits, id) for every logit of the row, in no particular order.  flush() runs after every group of up to eight
// logits handed to f (so that f can sum in fp32 and flush can fold the partial sum into a double).
template <int DT, class F, class G>
__device__ __forceinline__ void for_each_logit(const void* rowp, int V, F f, G flush) {
    for_each_vector<DT>(
        rowp, V,
        [&](const uint4& v, int i0) {
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                if (DT == PSMC_BF16) {
                    f(w[c] & 0xffffu, i0 + 2 * c);
                    f(w[c] >> 16, i0 + 2 * c + 1);
                } else {
                    f(w[c], i0 + c);
                }
            }
            flush();
        },
        f);
    flush();
}
template <int DT, class F>
__device__ __forceinline__ void for_each_logit(const void* rowp, int V, F f) {
    for_each_logit<DT>(rowp, V, f, [] {});
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

// One level of the search over candidates held in the shared-memory list: entries whose key matches the prefix so far
// (level 0 has no prefix to match).
template <int DT, int MODE>
__device__ __forceinline__ void count_list_level(const unsigned long long* list, int n_list, int level, uint32_t prefix,
                                                 bool nucleus, float neg_C, float bf, uint32_t* cnt,
                                                 unsigned long long* mass, int lane) {
    constexpr int kKeyBits = DT == PSMC_BF16 ? 16 : 32;
    const int shift = kKeyBits - 8 * (level + 1);
    for (int j = threadIdx.x; j < n_list; j += blockDim.x) {
        const uint32_t b = (uint32_t)list[j];
        const uint32_t key = key_of<DT>(b);
        if (level > 0 && (key >> (shift + 8)) != prefix) continue;
        const uint32_t d = (key >> shift) & 255u;
        atomicAdd(&cnt[d * 32 + lane], 1u);
        if (nucleus)
            atomicAdd(&mass[d * 16 + (lane & 15)],
                      __float2ull_rn(logit_mass<MODE>(value_of<DT>(b), neg_C, bf) * kFixOne));
    }
}

// Sum the [digit][lane] columns into per-digit totals (every thread of the CTA calls this; ends on a barrier).
__device__ __forceinline__ void fold_columns(const uint32_t* cnt, const unsigned long long* mass, bool nucleus,
                                             uint32_t* tot_cnt, unsigned long long* tot_mass) {
    __syncthreads();
    for (int d = threadIdx.x; d < kDigits; d += blockDim.x) {
        uint32_t c = 0;
        unsigned long long m = 0;
        for (int j = 0; j < 32; ++j) {  // thread d starts at column d, so the threads of a warp read different banks
            const int col = (j + d) & 31;
            c += cnt[d * 32 + col];
            if (nucleus && j < 16) m += mass[d * 16 + (col & 15)];
        }
        tot_cnt[d] = c;
        tot_mass[d] = m;
    }
    __syncthreads();
}
__device__ __forceinline__ void clear_columns(uint32_t* cnt, unsigned long long* mass, bool nucleus) {
    for (int i = threadIdx.x; i < kDigits * 32; i += blockDim.x) {
        cnt[i] = 0;
        if (nucleus && i < kDigits * 16) mass[i] = 0;
    }
    __syncthreads();
}

// Ascending bitonic sort of n2 (a power of two) 64-bit words in shared memory by the whole CTA.
// 128 words, four per lane (word e sits in lane e / 4, place e % 4), sorted ascending by one warp: a bitonic network
// whose exchanges run inside a lane for the two smallest strides and through shuffles otherwise.  No shared memory, no
// CTA barrier.
constexpr int kWarpList = 128;
__device__ __forceinline__ void warp_sort_128(unsigned long long (&v)[4], int lane) {
#pragma unroll
    for (int size = 2; size <= kWarpList; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride >= 1; stride >>= 1) {
            if (stride >= 4) {
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int e = lane * 4 + r;
                    const unsigned long long other = __shfl_xor_sync(kFull, v[r], stride >> 2);
                    const bool up = (e & size) == 0, low = (e & stride) == 0;  // ascending run; this is the lower index
                    const bool take_min = up == low;
                    v[r] = take_min ? (v[r] < other ? v[r] : other) : (v[r] > other ? v[r] : other);
                }
            } else {
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    if ((r & stride) == 0) {
                        const int e = lane * 4 + r;
                        const bool up = (e & size) == 0;
                        const unsigned long long a = v[r], b = v[r | stride];
                        const bool swap = up ? a > b : a < b;
                        v[r] = swap ? b : a;
                        v[r | stride] = swap ? a : b;
                    }
                }
            }
        }
    }
}

__device__ __forceinline__ void sort_words(unsigned long long* a, int n2) {
    for (int k = 2; k <= n2; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = threadIdx.x; i < n2; i += blockDim.x) {
                const int o = i ^ j;
                if (o > i) {
                    const unsigned long long x = a[i], y = a[o];
                    const bool up = (i & k) == 0;
                    if ((x > y) == up) {
                        a[i] = y;
                        a[o] = x;
                    }
                }
            }
            __syncthreads();
        }
    }
}

// What is left of a row once a short candidate list stands behind a top-k threshold, by ONE warp (see the call).
template <int DT, int MODE>
__device__ __noinline__ void finish_short_list(const MaskedParams& p, const unsigned long long* list, int n_cands, int k_top,
                                               const void* rowp, float C, double U, double S1, int row, int lane) {
    const float neg_C = -C;
    unsigned long long v[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int e = lane * 4 + r;
        v[r] = ~0ull;
        if (e < n_cands) {  // larger key first, lower id first among equal keys
            const unsigned long long w = list[e];
            v[r] = ((unsigned long long)(~key_of<DT>((uint32_t)w)) << 32) | (w >> 32);
        }
    }
    __syncwarp();  // the list has been read: its memory takes the ranked entries' payload below
    // (the rank order loses the logit's bits: keep them beside the id by sorting (rank word, bits) pairs would
    // need 96 bits; instead the bits are fetched again by id from the row after the second sort)
    warp_sort_128(v, lane);
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int e = lane * 4 + r;
        v[r] = e < k_top ? (v[r] & 0xffffffffull) : ~0ull;  // members of S by id; the rest sink to the end
    }
    warp_sort_128(v, lane);  // vocabulary order
    double m[4], mine = 0.0;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int e = lane * 4 + r;
        m[r] = e < k_top ? (double)logit_mass<MODE>(load_elem<DT>(rowp, (int)v[r]), neg_C, p.bf) : 0.0;
        mine += m[r];
    }
    const double incl = warp_scan_incl(mine, lane);
    const double Sb = __shfl_sync(kFull, incl, 31), target = U * Sb;
    const unsigned hit = __ballot_sync(kFull, mine > 0.0 && incl >= target);
    const unsigned has = __ballot_sync(kFull, mine > 0.0);
    if (!has) {  // no member of S has mass: cannot happen while the row's largest logit is in S
        if (lane == 0) {
            raise_status(p.status, PSMC_E_NUMERIC);
            p.tok[row] = -1;
            p.logp[row] = 0.0;
            p.loginc[row] = 0.0;
            p.set_size[row] = k_top;
        }
        return;
    }
    const int owner = hit ? __ffs(hit) - 1 : 31 - __clz(has);
    if (lane != owner) return;
    double run = incl - mine;
    int y = -1, last = -1;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        run += m[r];
        if (m[r] > 0.0) {
            last = (int)v[r];
            if (y < 0 && run >= target) y = last;
        }
    }
    if (y < 0) y = last;
    const double dl = (double)load_elem<DT>(rowp, y) - (double)C * kLn2;
    double add_s1, add_sb;
    ln_sum_corrections<MODE>(p.beta, add_s1, add_sb);
    const double ln_s1 = log(S1) + add_s1, ln_sb = log(Sb) + add_sb;
    p.tok[row] = y;
    p.logp[row] = dl - ln_s1;
    p.loginc[row] = (p.alpha_t - p.beta) * dl - p.alpha_t * ln_s1 + ln_sb;
    p.set_size[row] = k_top;
}

template <int DT, int MODE>
__global__ void __launch_bounds__(1024, 1) masked_rows_kernel(const __grid_constant__ MaskedParams p) {
    extern __shared__ __align__(16) unsigned char hist_raw[];
    const bool nucleus = p.top_k == 0;
    uint32_t* cnt = reinterpret_cast<uint32_t*>(hist_raw);                                      // [256][32]
    unsigned long long* mass = reinterpret_cast<unsigned long long*>(hist_raw + kCountBytes);  // [256][16], nucleus only
    unsigned long long* list =                                                                  // [kListCap] id << 32 | bits
        reinterpret_cast<unsigned long long*>(hist_raw + kCountBytes + (nucleus ? kMassBytes : 0));
    __shared__ double red[33];
    __shared__ uint32_t redu[64];
    __shared__ int redi[33];
    __shared__ uint32_t tot_cnt[kDigits];
    __shared__ unsigned long long tot_mass[kDigits];
    __shared__ Selection sel, thr;
    __shared__ double wmass[32];
    __shared__ int wties[32];
    __shared__ int n_list_sh, first_hit, last_mass;

    constexpr int kKeyBits = DT == PSMC_BF16 ? 16 : 32, kLevels = kKeyBits / 8;
    const int row = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const int V = p.V;
    chain_begin();
    if (p.zero_words && blockIdx.x == 0 && threadIdx.x < 2) p.zero_words[threadIdx.x] = 0;
    if (p.done[row]) return;
    const void* rowp = reinterpret_cast<const char*>(p.logits) + (size_t)row * p.ld * (DT == PSMC_F32 ? 4 : 2);
    const int g = row / p.N;
    const double U = hash_uniform(hash5(p.seed, kStreamToken, (uint64_t)g, (uint64_t)p.t, (uint64_t)(row - g * p.N)));

    if (threadIdx.x == 0) {
        sel.prefix = 0;
        sel.k_rem = (uint32_t)min(p.top_k, V);
        sel.m_rem = 0;
        sel.above = 0;
        n_list_sh = 0;
        first_hit = 0x7fffffff;
        last_mass = -1;
    }
    if (threadIdx.x < kDigits) tot_mass[threadIdx.x] = 0;  // read (and ignored) by the digit search when nothing weighs
    // (a thread's share is itself cut into kSub interleaved sub-shares, by position inside the 16-byte vectors)
    constexpr int kSub = DT == PSMC_BF16 ? 8 : 4;
    const bool by_threshold = !nucleus && 2 * p.top_k <= kSub * (int)blockDim.x;
    // A nucleus of share top_p < 1 holds no token of mass below (1 - top_p) / V of the row's: all such tokens together
    // stay under 1 - top_p, so the tokens above the floor already reach top_p.  The floor turns into a threshold on the
    // logit once the row's mass is known, and the search runs on the (usually short) list of tokens above it.
    const bool by_floor = nucleus && p.top_p <= 0.9999;  // (closer to 1 the slack of the argument drowns in rounding)
    if (by_threshold || by_floor) __syncthreads();
    else clear_columns(cnt, mass, nucleus);

    // ---- sweep 1: the row's largest logit; NaN and +inf make the row unusable; top-k by counting: first-level counts ----
    constexpr int kShift0 = kKeyBits - 8;
    // (on keys: a NaN or +inf ranks at or above +inf's key, or below -inf's)
    constexpr uint32_t kPosInf = DT == PSMC_BF16 ? 0xff80u : 0xff800000u, kNegInf = DT == PSMC_BF16 ? 0x007fu : 0x007fffffu;
    uint32_t kmax = 0u, kmin = 0xffffffffu;
    uint32_t sub[kSub];  // largest key of each sub-share (threshold path)
#pragma unroll
    for (int j = 0; j < kSub; ++j) sub[j] = 0u;
    if (DT == PSMC_BF16 && (by_threshold || by_floor)) {  // nothing to count: two keys at a time, packed maxima and minima
        constexpr uint32_t kNegInf2 = 0xff80ff80u;
        uint32_t mx2[4] = {kNegInf2, kNegInf2, kNegInf2, kNegInf2};
        for_each_vector<DT>(
            rowp, V,
            [&](const uint4& v, int) {
                mx2[0] = max_nan_pair(mx2[0], v.x);
                mx2[1] = max_nan_pair(mx2[1], v.y);
                mx2[2] = max_nan_pair(mx2[2], v.z);
                mx2[3] = max_nan_pair(mx2[3], v.w);
            },
            [&](uint32_t b, int) {
                const uint32_t key = key_of<DT>(b);
                kmax = max(kmax, key);
                kmin = min(kmin, key);
            });
#pragma unroll
        for (int c = 0; c < 4; ++c) {  // (a NaN maximum has the sign bit clear: its key ranks above +inf's)
            sub[(2 * c) % kSub] = key_of<DT>(mx2[c] & 0xffffu);
            sub[(2 * c + 1) % kSub] = key_of<DT>(mx2[c] >> 16);
        }
        sub[0] = max(sub[0], kmax);  // the ragged ends join the first sub-share
    } else if (by_threshold) {
        for_each_vector<DT>(
            rowp, V,
            [&](const uint4& v, int) {
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    if (DT == PSMC_BF16) {
                        const uint32_t a = key_of<DT>(w[c] & 0xffffu), b = key_of<DT>(w[c] >> 16);
                        sub[(2 * c) % kSub] = max(sub[(2 * c) % kSub], a);
                        sub[(2 * c + 1) % kSub] = max(sub[(2 * c + 1) % kSub], b);
                        kmin = min(kmin, min(a, b));
                    } else {
                        const uint32_t a = key_of<DT>(w[c]);
                        sub[c % kSub] = max(sub[c % kSub], a);
                        kmin = min(kmin, a);
                    }
                }
            },
            [&](uint32_t b, int) {
                const uint32_t key = key_of<DT>(b);
                sub[0] = max(sub[0], key);
                kmin = min(kmin, key);
            });
    } else {
        for_each_logit<DT>(rowp, V, [&](uint32_t b, int) {
            const uint32_t key = key_of<DT>(b);
            kmax = max(kmax, key);
            kmin = min(kmin, key);
            if (!nucleus) atomicAdd(&cnt[(key >> kShift0) * 32 + lane], 1u);
        });
    }
#pragma unroll
    for (int j = 0; j < kSub; ++j) kmax = max(kmax, sub[j]);
    kmax = __reduce_max_sync(kFull, kmax);
    kmin = __reduce_min_sync(kFull, kmin);
    if (lane == 0) {
        redu[warp] = kmax;
        redu[32 + warp] = kmin;
    }
    __syncthreads();
    for (int w = 0; w < nw; ++w) {
        kmax = max(kmax, redu[w]);
        kmin = min(kmin, redu[32 + w]);
    }
    const bool bad = kmax >= kPosInf || kmin < kNegInf;
    const float mx = value_of<DT>(bits_of_key<DT>(kmax));
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
    const float C = ref_exponent(mx, ref_shift(p.bf)), neg_C = -C;

    bool have_list = false;
    int first_list_level = 2;
    double s1 = 0.0;
    uint32_t prefix = 0;
    auto append = [&](uint32_t b, int i) {
        const int pos = atomicAdd(&n_list_sh, 1);
        if (pos < kListCap) list[pos] = ((unsigned long long)(uint32_t)i << 32) | b;
    };

    // the logits of one 16-byte vector (bf16) that are >= the threshold's go to the list: one test for all eight first
    auto collect8 = [&](const uint32_t (&w)[4], int i0, uint32_t th2) {
        const uint32_t g0 = ge_pair(w[0], th2), g1 = ge_pair(w[1], th2), g2 = ge_pair(w[2], th2), g3 = ge_pair(w[3], th2);
        if ((g0 | g1) | (g2 | g3)) {
            const uint32_t ge[4] = {g0, g1, g2, g3};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                if (ge[c] & 0xffffu) append(w[c] & 0xffffu, i0 + 2 * c);
                if (ge[c] >> 16) append(w[c] >> 16, i0 + 2 * c + 1);
            }
        }
    };

    if (by_threshold) {
        // ---- the threshold: the k-th largest of the threads' maxima, by the same digit search on a plain histogram ----
        if (threadIdx.x == 0) {
            thr.prefix = 0;
            thr.k_rem = (uint32_t)min(p.top_k, V);
            thr.m_rem = 0;
            thr.above = 0;
        }
        for (int level = 0; level < kLevels; ++level) {
            const int shift = kKeyBits - 8 * (level + 1);
            if (threadIdx.x < kDigits) tot_cnt[threadIdx.x] = 0;
            __syncthreads();
#pragma unroll
            for (int j = 0; j < kSub; ++j)
                if (level == 0 || (sub[j] >> (shift + 8)) == thr.prefix) atomicAdd(&tot_cnt[(sub[j] >> shift) & 255u], 1u);
            __syncthreads();
            if (warp == 0) pick_digit(thr, tot_cnt, tot_mass, false, false, level == kLevels - 1, 0.0, lane);
            __syncthreads();
        }
        const uint32_t theta = thr.prefix;
        // ---- sweep 2: the normaliser of p, and every logit at or above the threshold into the list ----
        if (DT == PSMC_BF16) {
            const uint32_t th2 = pair_threshold(theta);
            // (the packed fp32 arithmetic of the plain logit pass: both logits of a word at once, the same operations)
            const PackedConsts kc = packed_consts(p.bf);
            const f32x2 nc2 = pack2(neg_C, neg_C);
            for_each_vector<DT>(
                rowp, V,
                [&](const uint4& v, int i0) {
                    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
                    f32x2 part2 = ex2_2(rel_exponent2(widen_bf16x2(w[0]), nc2, kc));
#pragma unroll
                    for (int c = 1; c < 4; ++c) part2 = add2(part2, ex2_2(rel_exponent2(widen_bf16x2(w[c]), nc2, kc)));
                    const float2 part = unpack2(part2);
                    s1 += (double)(part.x + part.y);
                    collect8(w, i0, th2);
                },
                [&](uint32_t b, int i) {
                    s1 += (double)ex2(rel_exponent(value_of<DT>(b), neg_C));
                    if (key_of<DT>(b) >= theta) append(b, i);
                });
        } else {
            float part = 0.f;
            for_each_logit<DT>(
                rowp, V,
                [&](uint32_t b, int i) {
                    part += ex2(rel_exponent(value_of<DT>(b), neg_C));
                    if (key_of<DT>(b) >= theta) append(b, i);
                },
                [&] {
                    s1 += (double)part;
                    part = 0.f;
                });
        }
        __syncthreads();
        if (n_list_sh <= kListCap) {
            have_list = true;
            first_list_level = 0;
        } else {  // a crowd at the threshold (a row of equal logits, say): count digits after all
            __syncthreads();
            if (threadIdx.x == 0) n_list_sh = 0;
            s1 = 0.0;
            clear_columns(cnt, mass, nucleus);
            for_each_logit<DT>(rowp, V, [&](uint32_t b, int) { atomicAdd(&cnt[(key_of<DT>(b) >> kShift0) * 32 + lane], 1u); });
        }
    }

    bool m_rem_preset = false;
    if (by_floor) {
        // ---- sweep 2: the masses of p and of the proposal over the whole row ----
        double sb = 0.0;
        float part1 = 0.f, partb = 0.f;
        for_each_logit<DT>(
            rowp, V,
            [&](uint32_t b, int) {
                const float d = rel_exponent(value_of<DT>(b), neg_C);
                part1 += ex2(d);
                partb += mass_beta<MODE>(d, p.bf);
            },
            [&] {
                s1 += (double)part1;
                sb += (double)partb;
                part1 = 0.f;
                partb = 0.f;
            });
        const double Sb_row = block_sum(sb, red, nw);
        // floor on the mass, halved to stay on the safe side of rounding: 2^{beta (x - C)} >= (1 - top_p) Sb / (2 V)
        const double x_floor = (double)C + log2((1.0 - p.top_p) * Sb_row / (2.0 * (double)V)) / p.beta;
        float l_floor = (float)(x_floor * kLn2);
        l_floor = nextafterf(l_floor, -INFINITY);
        // a key at or below every key whose logit is >= l_floor (for bf16: the fp32 key's leading 16 bits)
        const uint32_t key32 = key_of<PSMC_F32>(__float_as_uint(l_floor));
        const uint32_t floor_key = (l_floor != l_floor || l_floor == -INFINITY) ? 0u
                                   : (DT == PSMC_BF16 ? key32 >> 16 : key32);
        // ---- sweep 3: the tokens at or above the floor into the list ----
        if (DT == PSMC_BF16) {
            const uint32_t th2 = pair_threshold(floor_key);
            for_each_vector<DT>(
                rowp, V,
                [&](const uint4& v, int i0) {
                    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
                    collect8(w, i0, th2);
                },
                [&](uint32_t b, int i) {
                    if (key_of<DT>(b) >= floor_key) append(b, i);
                });
        } else {
            for_each_logit<DT>(rowp, V, [&](uint32_t b, int i) {
                if (key_of<DT>(b) >= floor_key) append(b, i);
            });
        }
        __syncthreads();
        if (n_list_sh <= kListCap) {
            have_list = true;
            first_list_level = 0;
            m_rem_preset = true;  // the share is of the whole row's mass, not of the list's
            if (threadIdx.x == 0) {
                const double want = ceil(p.top_p * Sb_row * (double)kFixOne);
                sel.m_rem = want < 1.0 ? 1ull : (unsigned long long)want;
            }
        } else {  // a flat row: count digits and masses over the row after all
            __syncthreads();
            if (threadIdx.x == 0) n_list_sh = 0;
            s1 = 0.0;
            clear_columns(cnt, mass, nucleus);
        }
    }

    bool listed = have_list;
    if (!have_list) {
        // ---- sweep 2 (nucleus): first-level counts and masses, which need the reference exponent ----
        if (nucleus) {
            for_each_logit<DT>(rowp, V, [&](uint32_t b, int) {
                const uint32_t d = key_of<DT>(b) >> kShift0;
                atomicAdd(&cnt[d * 32 + lane], 1u);
                atomicAdd(&mass[d * 16 + (lane & 15)],
                          __float2ull_rn(logit_mass<MODE>(value_of<DT>(b), neg_C, p.bf) * kFixOne));
            });
        }
        fold_columns(cnt, mass, nucleus, tot_cnt, tot_mass);
        if (warp == 0) pick_digit(sel, tot_cnt, tot_mass, nucleus, true, kLevels == 1, p.top_p, lane);
        __syncthreads();
        prefix = sel.prefix;

        // ---- sweep 3: the second level (tokens whose first digit is the chosen one), and the normaliser of p ----
        constexpr int kShift1 = kKeyBits - 16;
        clear_columns(cnt, mass, nucleus);
        float part = 0.f;
        for_each_logit<DT>(
            rowp, V,
            [&](uint32_t b, int) {
                const float l = value_of<DT>(b);
                part += ex2(rel_exponent(l, neg_C));
                const uint32_t key = key_of<DT>(b);
                if ((key >> kShift0) != prefix) return;
                const uint32_t d = (key >> kShift1) & 255u;
                atomicAdd(&cnt[d * 32 + lane], 1u);
                if (nucleus)
                    atomicAdd(&mass[d * 16 + (lane & 15)], __float2ull_rn(logit_mass<MODE>(l, neg_C, p.bf) * kFixOne));
            },
            [&] {
                s1 += (double)part;
                part = 0.f;
            });
        fold_columns(cnt, mass, nucleus, tot_cnt, tot_mass);
        if (warp == 0) pick_digit(sel, tot_cnt, tot_mass, nucleus, false, kLevels == 2, p.top_p, lane);
        __syncthreads();
        prefix = sel.prefix;
        // tokens whose leading 16 key bits are at or above the 16 chosen so far: S, the ties at the cut, and (fp32)
        // the tokens that share the cut's leading bits
        listed = (int)(sel.above + tot_cnt[prefix & 255u]) <= kListCap;
        if (listed) {
            // ---- sweep 4: the candidates into the list ----
            const uint32_t cut = prefix << (kKeyBits - 16);
            for_each_logit<DT>(rowp, V, [&](uint32_t b, int i) {
                if (key_of<DT>(b) >= cut) append(b, i);
            });
        }
    }

    if (listed) {
        __syncthreads();
        const int n_cands = min(n_list_sh, kListCap);

        // ---- a short list behind a top-k threshold: everything that is left, by one warp and without CTA barriers ----
        // The general way below spends a dozen CTA barriers on a hundred entries (digit search, filter, sort, two
        // scans: 10 us of the 39 us a row took, with 15 of the 16 warps idle).  Here the candidates are ranked by
        // (logit descending, id ascending) in one sort -- the first k of that order are S, ties at the cut included --
        // then S is put in vocabulary order by a second sort, and the masses and the inverse CDF are warp scans.
        const int k_top = min(p.top_k, V);
        if (by_threshold && first_list_level == 0 && n_cands <= kWarpList && n_cands >= k_top) {
            const double S1 = block_sum(s1, red, nw);
            if (warp != 0) return;
            finish_short_list<DT, MODE>(p, list, n_cands, k_top, rowp, C, U, S1, row, lane);
            return;
        }

        // ---- the levels not yet decided, over the candidates in whatever order they arrived ----
        const bool short_list = n_cands <= 2 * (int)blockDim.x;  // few entries: no columns, one counter per digit
        for (int level = first_list_level; level < kLevels; ++level) {
            if (short_list) {
                if (threadIdx.x < kDigits) {
                    tot_cnt[threadIdx.x] = 0;
                    tot_mass[threadIdx.x] = 0;
                }
                __syncthreads();
                const int shift = kKeyBits - 8 * (level + 1);
                for (int j = threadIdx.x; j < n_cands; j += blockDim.x) {
                    const uint32_t b = (uint32_t)list[j], key = key_of<DT>(b);
                    if (level > 0 && (key >> (shift + 8)) != prefix) continue;
                    const uint32_t d = (key >> shift) & 255u;
                    atomicAdd(&tot_cnt[d], 1u);
                    if (nucleus)
                        atomicAdd(&tot_mass[d], __float2ull_rn(logit_mass<MODE>(value_of<DT>(b), neg_C, p.bf) * kFixOne));
                }
                __syncthreads();
            } else {
                clear_columns(cnt, mass, nucleus);
                count_list_level<DT, MODE>(list, n_cands, level, prefix, nucleus, neg_C, p.bf, cnt, mass, lane);
                fold_columns(cnt, mass, nucleus, tot_cnt, tot_mass);
            }
            if (warp == 0)
                pick_digit(sel, tot_cnt, tot_mass, nucleus, level == 0 && !m_rem_preset, level == kLevels - 1, p.top_p, lane);
            __syncthreads();
            prefix = sel.prefix;
        }
        const double S1 = block_sum(s1, red, nw);
        const uint32_t T = prefix, need = sel.need;
        const bool all_ties = need == sel.n_ties;
        const int set_size = (int)(sel.above + need);

        // ---- keep the candidates at or above the cut (S and the ties at T), sorted by token id ----
        // The counters are done with; their memory takes the second list.
        unsigned long long* kept = reinterpret_cast<unsigned long long*>(hist_raw);
        if (threadIdx.x == 0) n_list_sh = 0;
        __syncthreads();
        for (int j = threadIdx.x; j < n_cands; j += blockDim.x) {
            const unsigned long long w = list[j];
            if (key_of<DT>((uint32_t)w) >= T) kept[atomicAdd(&n_list_sh, 1)] = w;
        }
        __syncthreads();
        const int n_list = n_list_sh;  // = tokens above the cut + ties at it <= n_cands
        int n2 = 1;
        while (n2 < n_list) n2 <<= 1;
        for (int i = n_list + threadIdx.x; i < n2; i += blockDim.x) kept[i] = ~0ull;
        __syncthreads();
        sort_words(kept, n2);  // vocabulary order

        // ---- ordered part: thread t holds entries [e0, e1) of the sorted list ----
        const int E = (n_list + (int)blockDim.x - 1) / (int)blockDim.x;
        const int e0 = min(n_list, (int)threadIdx.x * E), e1 = min(n_list, e0 + E);
        int c = 0;
        for (int j = e0; j < e1; ++j) c += key_of<DT>((uint32_t)kept[j]) == T;
        const int tie_base = block_scan_incl(c, redi, (int*)nullptr, nw) - c;
        auto entry_mass = [&](unsigned long long w, int& rank) -> double {  // mass of an entry if it is in S, else 0
            const uint32_t b = (uint32_t)w, key = key_of<DT>(b);
            bool in = key > T;
            if (key == T) {
                in = all_ties || (uint32_t)rank < need;
                ++rank;
            }
            return in ? (double)logit_mass<MODE>(value_of<DT>(b), neg_C, p.bf) : 0.0;
        };
        double acc = 0.0;
        int rank = tie_base;
        for (int j = e0; j < e1; ++j) acc += entry_mass(kept[j], rank);
        double Sb;
        const double incl = block_scan_incl(acc, red, &Sb, nw);
        const double target = U * Sb;
        if (acc > 0.0) {
            if (incl >= target) atomicMin(&first_hit, (int)threadIdx.x);
            atomicMax(&last_mass, (int)threadIdx.x);
        }
        __syncthreads();
        const int owner = first_hit != 0x7fffffff ? first_hit : last_mass;
        if ((int)threadIdx.x != owner) {
            if (threadIdx.x == 0 && owner < 0) {  // no entry of S has mass: cannot happen while the largest logit is in S
                raise_status(p.status, PSMC_E_NUMERIC);
                p.tok[row] = -1;
                p.logp[row] = 0.0;
                p.loginc[row] = 0.0;
                p.set_size[row] = set_size;
            }
            return;
        }
        double run = incl - acc;
        int y = -1, last = -1;
        rank = tie_base;
        for (int j = e0; j < e1 && y < 0; ++j) {
            const double m = entry_mass(kept[j], rank);
            run += m;
            if (m > 0.0) {
                last = (int)(kept[j] >> 32);
                if (run >= target) y = last;
            }
        }
        if (y < 0) y = last;
        const double dl = (double)load_elem<DT>(rowp, y) - (double)C * kLn2;
        double add_s1, add_sb;
        ln_sum_corrections<MODE>(p.beta, add_s1, add_sb);  // both sums are made of ex2 terms, on the list as on the row
        const double ln_s1 = log(S1) + add_s1, ln_sb = log(Sb) + add_sb;
        p.tok[row] = y;
        p.logp[row] = dl - ln_s1;
        p.loginc[row] = (p.alpha_t - p.beta) * dl - p.alpha_t * ln_s1 + ln_sb;
        p.set_size[row] = set_size;
        return;
    }

    // ---- too many candidates for the list: every remaining step sweeps the row ----
    for (int level = 2; level < kLevels; ++level) {
        const int shift = kKeyBits - 8 * (level + 1);
        clear_columns(cnt, mass, nucleus);
        for_each_logit<DT>(rowp, V, [&](uint32_t b, int) {
            const uint32_t key = key_of<DT>(b);
            if ((key >> (shift + 8)) != prefix) return;
            const uint32_t d = (key >> shift) & 255u;
            atomicAdd(&cnt[d * 32 + lane], 1u);
            if (nucleus)
                atomicAdd(&mass[d * 16 + (lane & 15)],
                          __float2ull_rn(logit_mass<MODE>(value_of<DT>(b), neg_C, p.bf) * kFixOne));
        });
        fold_columns(cnt, mass, nucleus, tot_cnt, tot_mass);
        if (warp == 0) pick_digit(sel, tot_cnt, tot_mass, nucleus, false, level == kLevels - 1, p.top_p, lane);
        __syncthreads();
        prefix = sel.prefix;
    }
    const double S1 = block_sum(s1, red, nw);
    const uint32_t T = prefix, need = sel.need;
    const bool all_ties = need == sel.n_ties;
    const int set_size = (int)(sel.above + need);

    // Ordered sweeps: warp w owns logits [lo, hi); in a round its lanes take kPer consecutive logits each (one 16-byte
    // load where the row allows), so a round covers 32 * kPer logits in id order: lane 0's first.
    constexpr int kPer = DT == PSMC_BF16 ? 8 : 4;
    const bool aligned = (reinterpret_cast<uintptr_t>(rowp) & 15) == 0;
    const int seg = (((V + nw - 1) / nw) + 32 * kPer - 1) / (32 * kPer) * (32 * kPer);
    const int lo = min(V, warp * seg), hi = min(V, lo + seg);
    auto load_chunk = [&](int e0, uint32_t (&bits)[kPer]) -> int {  // -> how many of the kPer logits from e0 exist
        if (e0 >= hi) return 0;
        if (aligned && e0 + kPer <= hi) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(rowp) +
                                                                 (size_t)e0 * (DT == PSMC_BF16 ? 2 : 4)));
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                if (DT == PSMC_BF16) {
                    bits[2 * c] = w[c] & 0xffffu;
                    bits[2 * c + 1] = w[c] >> 16;
                } else {
                    bits[c] = w[c];
                }
            }
            return kPer;
        }
        const int nv = min(kPer, hi - e0);
#pragma unroll
        for (int j = 0; j < kPer; ++j) bits[j] = j < nv ? load_bits<DT>(rowp, e0 + j) : 0u;
        return nv;
    };
    int tie_base = 0;
    if (!all_ties) {  // ties at T are taken in id order: how many lie before this warp's stretch
        int n = 0;
        for (int base = lo; base < hi; base += 32 * kPer) {
            uint32_t bits[kPer];
            const int nv = load_chunk(base + lane * kPer, bits);
#pragma unroll
            for (int j = 0; j < kPer; ++j) n += (j < nv && key_of<DT>(bits[j]) == T) ? 1 : 0;
        }
        n = warp_scan_incl(n, lane);
        if (lane == 31) wties[warp] = n;
        __syncthreads();
        for (int w = 0; w < warp; ++w) tie_base += wties[w];
    }
    // masses of this lane's logits that are in S; `rank` = ties at T before them in the row
    auto chunk_masses = [&](const uint32_t (&bits)[kPer], int nv, int rank, double (&m)[kPer]) -> double {
        double sum = 0.0;
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            m[j] = 0.0;
            if (j < nv) {
                const uint32_t key = key_of<DT>(bits[j]);
                bool in = key > T;
                if (key == T) {
                    in = all_ties || (uint32_t)rank < need;
                    ++rank;
                }
                if (in) m[j] = (double)logit_mass<MODE>(value_of<DT>(bits[j]), neg_C, p.bf);
                sum += m[j];
            }
        }
        return sum;
    };
    auto ties_before_lane = [&](const uint32_t (&bits)[kPer], int nv, int& tb) -> int {  // and advances tb by the round's ties
        if (all_ties) return 0;
        int c = 0;
#pragma unroll
        for (int j = 0; j < kPer; ++j) c += (j < nv && key_of<DT>(bits[j]) == T) ? 1 : 0;
        const int incl = warp_scan_incl(c, lane);
        const int rank = tb + incl - c;
        tb += __shfl_sync(kFull, incl, 31);
        return rank;
    };
    {
        double acc = 0.0;
        int tb = tie_base;
        for (int base = lo; base < hi; base += 32 * kPer) {
            uint32_t bits[kPer];
            double m[kPer];
            const int nv = load_chunk(base + lane * kPer, bits);
            const int rank = ties_before_lane(bits, nv, tb);
            acc += chunk_masses(bits, nv, rank, m);
        }
        acc = warp_sum(acc);
        if (lane == 0) wmass[warp] = acc;
    }
    __syncthreads();
    double Sb = 0.0;
    for (int w = 0; w < nw; ++w) Sb += wmass[w];
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

    // the warp that holds the target: the round, the lane, the token
    int y = -1, last_pos = -1;
    double run = run0;
    int tb = tie_base;
    for (int base = lo; base < hi && y < 0; base += 32 * kPer) {
        uint32_t bits[kPer];
        double m[kPer];
        const int e0 = base + lane * kPer;
        const int nv = load_chunk(e0, bits);
        const int rank = ties_before_lane(bits, nv, tb);
        const double e = chunk_masses(bits, nv, rank, m);
        const double incl = run + warp_scan_incl(e, lane);
        const unsigned hit = __ballot_sync(kFull, e > 0.0 && incl >= target);
        const unsigned pos = __ballot_sync(kFull, e > 0.0);
        const int src = hit ? __ffs(hit) - 1 : (pos ? 31 - __clz(pos) : -1);
        if (src >= 0) {  // lane src: its first logit that reaches the target, else its last one with mass
            int mine = -1;
            if (lane == src) {
                double r = incl - e;
                int last = -1;
#pragma unroll
                for (int j = 0; j < kPer; ++j) {
                    if (m[j] > 0.0) {
                        r += m[j];
                        last = e0 + j;
                        if (mine < 0 && hit && r >= target) mine = last;
                    }
                }
                if (mine < 0) mine = last;
            }
            mine = __shfl_sync(kFull, mine, src);
            if (hit) y = mine;
            else last_pos = mine;
        }
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
            double add_s1, add_sb;
            ln_sum_corrections<MODE>(p.beta, add_s1, add_sb);
            const double ln_s1 = log(S1) + add_s1, ln_sb = log(Sb) + add_sb;
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

// the per-group update from row results that a kernel before it on the stream left in memory
cudaError_t launch_rows_weights(const WeightsArgs& wa, cudaStream_t stream) {
    const int warps = (wa.N + 31) / 32;
    return launch_chained(rows_weights_kernel, dim3((unsigned)wa.G), dim3((unsigned)(warps * 32)), 0, stream, wa);
}

cudaError_t launch_step_masked(const LogitsStreamArgs& la, const WeightsArgs& wa, int top_k, double top_p,
                               int32_t* set_size, cudaStream_t stream) {
    MaskedParams p;
    p.logits = la.logits; p.V = la.V; p.ld = la.ld; p.N = wa.N; p.t = wa.t; p.top_k = top_k; p.top_p = top_p;
    p.beta = wa.beta; p.alpha_t = wa.alpha_t; p.bf = (float)wa.beta; p.seed = wa.seed; p.done = la.done;
    p.tok = wa.tok; p.logp = wa.logp; p.loginc = wa.loginc; p.set_size = set_size; p.zero_words = la.zero_words;
    p.status = la.status;
    const int mode = beta_mode(wa.beta);
    MaskedFn fn = la.dt == PSMC_F32 ? pick_masked<PSMC_F32>(mode) : pick_masked<PSMC_BF16>(mode);
    const size_t smem = (size_t)kCountBytes + (top_k == 0 ? kMassBytes : 0) + (size_t)kListCap * 8;
    cudaError_t e = allow_dynamic_smem(reinterpret_cast<const void*>(fn), kCountBytes + kMassBytes + kListCap * 8);
    if (e != cudaSuccess) return e;
    const int threads = la.V < 16384 ? 256 : 512;
    e = launch_chained(fn, dim3((unsigned)la.R), dim3((unsigned)threads), smem, stream, p);
    if (e != cudaSuccess) return e;
    return launch_rows_weights(wa, stream);
}

}  // namespace psmc
