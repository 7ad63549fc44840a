// KV-cache reindex (the cache reorder of Algorithm 1's resampling branch, Appendix C): copy the live prefix of surviving rows
// onto the rows of discarded particles, for every layer, K and V, and head.
//
// The move list comes from the resampling kernel as "sources": one record per surviving row
// with surplus offspring, naming the rows that receive it.  A source chunk is read ONCE and
// written to each of its destinations, so bytes moved = unique reads + writes.
//
// Bulk path (sm_100a): one warp per CTA; lane 0 drives a ring of shared-memory stages with the
// TMA engine: cp.async.bulk global->shared (completion on an mbarrier), then cp.async.bulk
// shared->global per destination (bulk async-groups).  No thread touches the payload, so the copy
// is bit-exact by construction and the SM's load/store units stay idle.
// Every mbarrier wait is bounded; on expiry the kernel raises PSMC_E_TIMEOUT, drains its own
// copies and returns.  Plain path: 256 threads copy with ordinary loads/stores of the widest unit
// the alignment allows; used when the 16-byte rules of bulk copies do not hold.
#include "bulk_copy.cuh"
#include "common.cuh"
#include "internal.h"

namespace psmc {
namespace {

constexpr int kChunk = 16384;   // bytes per stage
constexpr int kStages = 4;
constexpr int kBulkCtasPerSm = 3;
constexpr int kUnitParts = 4;   // a (source, tensor, head) segment is handed out in this many parts (whole chunks each)
// Work is handed out in units of a quarter of one (source record, pointer/head segment): the live prefix of one head
// of one K or V tensor of one surviving row, cut at chunk boundaries.  Lengths differ from row to row, so a static
// deal of fixed-size pieces leaves CTAs with unequal loads; instead every CTA takes the next unit from a global
// counter when it runs out (the fetch of the unit after that is already in flight, so its latency stays off the copy
// pipeline).  The last unit a CTA draws is what the others wait for at the end of the kernel: with whole segments
// (180 KB at 700 positions, read once and written 2-3 times) that tail was 4-5 % of the kernel.
// A unit is streamed in chunks of kChunk bytes.
struct Item {
    const char* src;
    int64_t dst_off;  // byte offset inside a destination row-head segment = chunk * kChunk
    int seg_ptr, seg_head;
    int dst_begin, n_dst;
    uint32_t bytes;
};
struct UnitCursor {
    int seg_ptr, seg_head, dst_begin, n_dst;
    const char* src;     // start of the source segment
    int64_t seg_bytes;   // live bytes of the segment
    int64_t off;         // next byte to hand out
};
__device__ __forceinline__ void open_unit(const KvLaunch& k, int u, int n_seg, UnitCursor& c) {
    const int part = u % kUnitParts, us = u / kUnitParts;
    const int s = us / n_seg, seg = us - s * n_seg;
    const MoveSource ms = k.sources[s];
    const int len = ms.len < k.max_len ? ms.len : k.max_len;
    int skip = k.skip_pos ? k.skip_pos[ms.src_row / k.N] : 0;  // a prompt shared by the group stays where it is
    skip = skip < 0 ? 0 : (skip > len ? len : skip);
    c.seg_ptr = seg / k.H;
    c.seg_head = seg - c.seg_ptr * k.H;
    c.dst_begin = ms.dst_begin;
    c.n_dst = ms.n_dst;
    c.src = k.src[c.seg_ptr] + (int64_t)ms.src_row * k.row_bytes_stride + (int64_t)c.seg_head * k.head_bytes_stride;
    // the part's share of [skip, len): whole chunks, the last part takes the ragged end
    const int64_t lo = (int64_t)skip * k.pos_bytes, hi = (int64_t)(len > 0 ? len : 0) * k.pos_bytes;
    const int64_t chunks = (hi - lo + kChunk - 1) / kChunk, per_part = (chunks + kUnitParts - 1) / kUnitParts;
    const int64_t p_lo = lo + (int64_t)part * per_part * kChunk, p_hi = p_lo + per_part * kChunk;
    c.off = p_lo < hi ? p_lo : hi;
    c.seg_bytes = p_hi < hi ? p_hi : hi;  // the cursor runs from off to seg_bytes
}
__device__ __forceinline__ void take_chunk(UnitCursor& c, Item& it) {
    it.src = c.src + c.off;
    it.dst_off = c.off;
    it.seg_ptr = c.seg_ptr;
    it.seg_head = c.seg_head;
    it.dst_begin = c.dst_begin;
    it.n_dst = c.n_dst;
    const int64_t left = c.seg_bytes - c.off;
    it.bytes = (uint32_t)(left < kChunk ? left : kChunk);
    c.off += it.bytes;
}
__device__ __forceinline__ char* dst_addr(const KvLaunch& k, const Item& it, int d) {
    const int row = k.dst_rows[it.dst_begin + d];
    return k.dst[it.seg_ptr] + (int64_t)row * k.dst_row_bytes_stride + (int64_t)it.seg_head * k.dst_head_bytes_stride +
           it.dst_off;
}
// Last CTA out puts the unit counter back to zero for the next launch (launches on one context are stream-ordered).
__device__ __forceinline__ void leave_queue(int32_t* work) {
    __threadfence();
    if (atomicInc(reinterpret_cast<unsigned int*>(work + 1), gridDim.x - 1) == gridDim.x - 1) {
        work[0] = 0;
        __threadfence();
    }
}

__global__ void __launch_bounds__(32) reindex_bulk_kernel(const __grid_constant__ KvLaunch k) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t bars[kStages];
    __shared__ Item ring[kStages];

    chain_begin();
    const int n_src = *reinterpret_cast<const volatile int32_t*>(k.n_sources);
    if (n_src <= 0) return;  // nothing resampled this step
    if (threadIdx.x != 0) return;

    for (int s = 0; s < kStages; ++s) mbar_init(&bars[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();

    const int n_seg = k.n_ptrs * k.H;
    const int n_units = n_src * n_seg * kUnitParts;   // < 2^31: checked by the host (rows, pointers and heads per launch)

    // unit queue: `next_u` is always one fetch ahead of the unit being streamed
    UnitCursor cur;
    cur.seg_bytes = 0;
    cur.off = 0;
    int next_u = atomicAdd(k.work, 1);
    Item cand;
    auto advance = [&]() -> bool {  // next chunk into `cand`; false when the queue is dry
        while (cur.off >= cur.seg_bytes) {
            if (next_u >= n_units) return false;
            open_unit(k, next_u, n_seg, cur);
            next_u = atomicAdd(k.work, 1);
        }
        take_chunk(cur, cand);
        return true;
    };
    bool more = advance();

    int issued = 0, consumed = 0;
    bool failed = false;
    for (int i = 0;; ++i) {
        // consume item i-(kStages-1): its load has had kStages-1 iterations to land
        const int j = i - (kStages - 1);
        if (j >= 0 && j < issued) {
            const int slot = j % kStages;
            if (!mbar_wait(&bars[slot], (uint32_t)((j / kStages) & 1))) {
                failed = true;
                break;
            }
            fence_async_smem();
            const Item it = ring[slot];
            for (int d = 0; d < it.n_dst; ++d) bulk_store(dst_addr(k, it, d), smem + (size_t)slot * kChunk, it.bytes);
            bulk_commit();
            ++consumed;
        }
        // produce item i into slot i % kStages, last used by item i-kStages
        if (more) {
            const int slot = i % kStages;
            if (i >= kStages) bulk_wait_read<1>();  // all store groups but the newest have read their stage
            ring[slot] = cand;
            mbar_expect_tx(&bars[slot], cand.bytes);
            bulk_load(smem + (size_t)slot * kChunk, cand.src, cand.bytes, &bars[slot]);
            ++issued;
            more = advance();
        } else if (consumed == issued) {
            break;
        }
    }
    if (failed) {
        raise_status(k.status, PSMC_E_TIMEOUT);
        // do not leave with loads still landing in this CTA's shared memory: bounded second wait
        for (int j = consumed; j < issued; ++j) mbar_wait(&bars[j % kStages], (uint32_t)((j / kStages) & 1));
    }
    bulk_wait_all();
    leave_queue(k.work);
}

// ---- plain path: ordinary loads and stores of unit type U ----
template <typename U>
__global__ void __launch_bounds__(256) reindex_plain_kernel(const __grid_constant__ KvLaunch k) {
    __shared__ int sh_u;
    const int n_src = *reinterpret_cast<const volatile int32_t*>(k.n_sources);
    if (n_src <= 0) return;
    const int n_seg = k.n_ptrs * k.H;
    const int n_units = n_src * n_seg * kUnitParts;
    for (;;) {
        __syncthreads();  // everyone has read the previous sh_u
        if (threadIdx.x == 0) sh_u = atomicAdd(k.work, 1);
        __syncthreads();
        const int u = sh_u;
        if (u >= n_units) break;
        UnitCursor c;
        open_unit(k, u, n_seg, c);
        Item it;
        it.seg_ptr = c.seg_ptr; it.seg_head = c.seg_head; it.dst_begin = c.dst_begin; it.n_dst = c.n_dst; it.dst_off = 0;
        const int64_t n_units_u = c.seg_bytes / (int64_t)sizeof(U);
        const U* s = reinterpret_cast<const U*>(c.src);
        // four loads in flight per thread, then their stores (source and destination may lie in one tensor, so a plain
        // loop would wait for every load before the next store may go out)
        constexpr int kBatch = 4;
        for (int64_t e0 = c.off / (int64_t)sizeof(U) + threadIdx.x; e0 < n_units_u; e0 += (int64_t)kBatch * blockDim.x) {
            U v[kBatch];
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const int64_t e = e0 + (int64_t)u * blockDim.x;
                if (e < n_units_u) v[u] = s[e];
            }
            for (int d = 0; d < it.n_dst; ++d) {
                U* out = reinterpret_cast<U*>(dst_addr(k, it, d));
#pragma unroll
                for (int u = 0; u < kBatch; ++u) {
                    const int64_t e = e0 + (int64_t)u * blockDim.x;
                    if (e < n_units_u) out[e] = v[u];
                }
            }
        }
    }
    if (threadIdx.x == 0) leave_queue(k.work);
}

// ---- arbitrary gather vector -> move records, with the in-place hazard check ----
__global__ void __launch_bounds__(1024) build_moves_kernel(const int32_t* idx, int R, int max_len, int in_place,
                                                           MoveSource* sources, int32_t* dst_rows, int32_t* n_sources,
                                                           int32_t* n_moves, int32_t* status) {
    __shared__ int bad, count;
    if (threadIdx.x == 0) {
        bad = 0;
        count = 0;
    }
    __syncthreads();
    for (int kk = threadIdx.x; kk < R; kk += blockDim.x) {
        const int s = idx[kk];
        if (s < 0 || s >= R) {
            atomicMax(&bad, PSMC_E_INVAL);
        } else if (in_place && s != kk && idx[s] != s) {
            atomicMax(&bad, PSMC_E_HAZARD);  // row s is read here and rewritten elsewhere
        }
    }
    __syncthreads();
    if (bad) {
        if (threadIdx.x == 0) {
            *n_sources = 0;
            *n_moves = 0;
            raise_status(status, bad);
        }
        return;
    }
    for (int kk = threadIdx.x; kk < R; kk += blockDim.x) {
        const int s = idx[kk];
        if (in_place && s == kk) continue;
        const int pos = atomicAdd(&count, 1);
        dst_rows[pos] = kk;
        MoveSource ms;
        ms.src_row = s;
        ms.len = max_len;
        ms.dst_begin = pos;
        ms.n_dst = 1;
        sources[pos] = ms;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        *n_sources = count;
        *n_moves = count;
    }
}

}  // namespace

int reindex_unit_parts() { return kUnitParts; }

cudaError_t launch_reindex_kv(const KvLaunch& k, cudaStream_t stream) {
    if (k.bulk_ok) {
        const int smem = kStages * kChunk;
        cudaError_t e = allow_dynamic_smem(reinterpret_cast<const void*>(reindex_bulk_kernel), smem);
        if (e != cudaSuccess) return e;
        return launch_chained(reindex_bulk_kernel, dim3(kSMs * kBulkCtasPerSm), dim3(32), (size_t)smem, stream, k);
    }
    // widest unit that divides every address, stride and row size
    uint64_t bits = (uint64_t)k.row_bytes_stride | (uint64_t)k.head_bytes_stride | (uint64_t)k.dst_row_bytes_stride |
                    (uint64_t)k.dst_head_bytes_stride | (uint64_t)k.pos_bytes;
    for (int i = 0; i < k.n_ptrs; ++i) bits |= (uint64_t)(uintptr_t)k.src[i] | (uint64_t)(uintptr_t)k.dst[i];
    const int grid = kSMs * 8;
    if (bits % 16 == 0) reindex_plain_kernel<uint4><<<grid, 256, 0, stream>>>(k);
    else if (bits % 8 == 0) reindex_plain_kernel<uint2><<<grid, 256, 0, stream>>>(k);
    else if (bits % 4 == 0) reindex_plain_kernel<uint32_t><<<grid, 256, 0, stream>>>(k);
    else if (bits % 2 == 0) reindex_plain_kernel<uint16_t><<<grid, 256, 0, stream>>>(k);
    else reindex_plain_kernel<uint8_t><<<grid, 256, 0, stream>>>(k);
    return cudaGetLastError();
}

cudaError_t launch_build_moves(const int32_t* idx, int R, int max_len, int in_place, MoveSource* sources,
                               int32_t* dst_rows, int32_t* n_sources, int32_t* n_moves, int32_t* status,
                               cudaStream_t stream) {
    build_moves_kernel<<<1, 1024, 0, stream>>>(idx, R, max_len, in_place, sources, dst_rows, n_sources, n_moves, status);
    return cudaGetLastError();
}

}  // namespace psmc
