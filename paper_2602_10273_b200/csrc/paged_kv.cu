// Paged KV cache with copy-on-write resampling: the cache reorder of Algorithm 1's resampling branch / Appendix C carried out
// on a block table.  A rewritten slot gives its blocks back, takes a reference to every full block of its ancestor
// and a private copy of the ancestor's partly filled last block.  Position p of row r lives in block
// table[r][p / block_len] at offset p % block_len of pools laid out [n_blocks, H, block_len, D].
//
// Kernels (all tiny except the copy, which moves < block_len positions per rewritten slot):
//   paged_init_kernel      free list, tables, the blocks of the prompts (set-up, one CTA)
//   paged_append_kernel    a new block for every live row whose next position starts one (pops only)
//   paged_release_kernel   rewritten slots return their blocks (pushes only)
//   paged_acquire_kernel   table entries and reference counts of the ancestors' full blocks, a fresh block for
//                          the partly filled one (pops only); leaves one copy order per rewritten slot; then the
//                          append for the next token, so that a token costs three launches here, not four
//   paged_copy_kernel      the copy orders: (layer, K/V, head) x live positions of the last block
// Pushes and pops never meet in one kernel, so the free list needs nothing beyond one atomic counter.
#include "common.cuh"
#include "internal.h"

namespace psmc {
namespace {

struct CopyOrder {
    int32_t src_blk, dst_blk, positions;
};
// copy orders of the last reindex, one per rewritten slot (at the slot's place in the move list; positions = 0 when
// the ancestor has no partly filled block).  They live behind the free list, in the same allocation.
__device__ __forceinline__ CopyOrder* orders_of(const PagedState& ps) {
    return reinterpret_cast<CopyOrder*>(ps.free_list + ps.n_blocks);
}

// one block off the free list (kernels that only pop); -1 and the error code when there is none
__device__ __forceinline__ int pop_block(const PagedState& ps, int32_t* status) {
    const int idx = atomicSub(ps.free_top, 1);
    if (idx <= 0) {
        atomicAdd(ps.free_top, 1);
        raise_status(status, PSMC_E_NOMEM);
        return -1;
    }
    return ps.free_list[idx - 1];
}

__global__ void __launch_bounds__(1024) paged_init_kernel(const PagedState ps, const int32_t* prompt_len, int G,
                                                          int share_prompt, int32_t* status) {
    for (int i = threadIdx.x; i < ps.n_blocks; i += blockDim.x) {
        ps.refc[i] = 0;
        ps.free_list[i] = ps.n_blocks - 1 - i;  // popped from the top: blocks 0, 1, 2, ...
    }
    for (int64_t i = threadIdx.x; i < (int64_t)ps.R * ps.max_blocks; i += blockDim.x) ps.table[i] = -1;
    __syncthreads();
    if (threadIdx.x != 0) return;
    int top = ps.n_blocks;
    const int B = ps.block_len, N = ps.N;
    bool ok = true;
    auto pop = [&]() -> int {
        if (top <= 0) {
            ok = false;
            return -1;
        }
        return ps.free_list[--top];
    };
    for (int g = 0; g < G && ok; ++g) {
        const int P = prompt_len[g], nfull = P / B, rem = P % B;
        if (nfull + (rem ? 1 : 0) > ps.max_blocks) {
            ok = false;
            break;
        }
        if (share_prompt) {
            for (int j = 0; j < nfull && ok; ++j) {  // one block for the whole group
                const int blk = pop();
                if (blk < 0) break;
                ps.refc[blk] = N;
                for (int i = 0; i < N; ++i) ps.table[(int64_t)(g * N + i) * ps.max_blocks + j] = blk;
            }
        }
        for (int i = 0; i < N && ok; ++i) {
            const int64_t row = (int64_t)(g * N + i) * ps.max_blocks;
            for (int j = share_prompt ? nfull : 0; j < nfull + (rem ? 1 : 0) && ok; ++j) {  // private blocks
                const int blk = pop();
                if (blk < 0) break;
                ps.refc[blk] = 1;
                ps.table[row + j] = blk;
            }
        }
    }
    *ps.free_top = top;
    if (!ok) raise_status(status, PSMC_E_NOMEM);
}

// A block for row r's next position if that position starts a block and the row has none there yet (pops only).
__device__ __forceinline__ void append_row(const PagedState& ps, int r, const int32_t* len, const uint8_t* done,
                                           int32_t* status) {
    if (done[r]) return;
    const int p = len[r];
    if (p % ps.block_len != 0) return;  // the row's last block still has room
    const int j = p / ps.block_len;
    if (j >= ps.max_blocks) {
        raise_status(status, PSMC_E_STATE);
        return;
    }
    int32_t* slot = ps.table + (int64_t)r * ps.max_blocks + j;
    if (*slot >= 0) return;  // already there (an earlier call, or the reindex before this token)
    const int blk = pop_block(ps, status);
    if (blk < 0) return;
    ps.refc[blk] = 1;
    *slot = blk;
}

__global__ void paged_append_kernel(const PagedState ps, const int32_t* len, const uint8_t* done, int32_t* status) {
    chain_begin();
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r < ps.R) append_row(ps, r, len, done, status);
}

__global__ void paged_release_kernel(const PagedState ps, const int32_t* dst_rows, const int32_t* n_moves) {
    chain_begin();
    const int n = *n_moves;
    const int64_t total = (int64_t)n * ps.max_blocks;
    for (int64_t w = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; w < total; w += (int64_t)gridDim.x * blockDim.x) {
        const int m = (int)(w / ps.max_blocks), j = (int)(w - (int64_t)m * ps.max_blocks);
        int32_t* slot = ps.table + (int64_t)dst_rows[m] * ps.max_blocks + j;
        const int blk = *slot;
        if (blk < 0) continue;
        *slot = -1;
        if (atomicSub(&ps.refc[blk], 1) == 1) ps.free_list[atomicAdd(ps.free_top, 1)] = blk;  // last owner: back on the list
    }
}

// len / done non-NULL: the kernel also gives every live row the block its next position needs (what
// paged_append_kernel does), so that the next token needs no launch of its own for that.
__global__ void paged_acquire_kernel(const PagedState ps, const MoveSource* sources, const int32_t* dst_rows,
                                     const int32_t* n_sources, const int32_t* len, const uint8_t* done,
                                     int32_t* status) {
    chain_begin();
    const int n = *n_sources;
    CopyOrder* orders = orders_of(ps);
    const int lane = threadIdx.x & 31;
    const int warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, n_warps = (gridDim.x * blockDim.x) >> 5;
    // one warp per surviving source: its lanes share the full blocks (a reference per destination, the table entries of
    // every destination) and then the destinations (a fresh block each for the partly filled one)
    for (int s = warp_global; s < n; s += n_warps) {
        const MoveSource ms = sources[s];
        const int nfull = ms.len / ps.block_len, rem = ms.len % ps.block_len;
        const int32_t* src_row = ps.table + (int64_t)ms.src_row * ps.max_blocks;
        for (int j = lane; j < nfull; j += 32) {
            const int blk = src_row[j];
            if (blk >= 0) atomicAdd(&ps.refc[blk], ms.n_dst);
            else raise_status(status, PSMC_E_STATE);  // a live position without a block: the table was not kept up
            for (int d = 0; d < ms.n_dst; ++d)
                ps.table[(int64_t)dst_rows[ms.dst_begin + d] * ps.max_blocks + j] = blk;
        }
        const int last_blk = rem ? src_row[nfull] : -1;
        if (rem && last_blk < 0 && lane == 0) raise_status(status, PSMC_E_STATE);
        for (int d = lane; d < ms.n_dst; d += 32) {
            const int m = ms.dst_begin + d;
            CopyOrder o{-1, -1, 0};
            if (rem && last_blk >= 0) {
                const int blk = pop_block(ps, status);
                if (blk >= 0) {
                    ps.refc[blk] = 1;
                    ps.table[(int64_t)dst_rows[m] * ps.max_blocks + nfull] = blk;
                    o.src_blk = last_blk;
                    o.dst_blk = blk;
                    o.positions = rem;
                }
            }
            orders[m] = o;  // one order per rewritten slot, at the slot's place in the move list
        }
    }
    // The next token's blocks.  A rewritten slot's entry for a block that starts at its length is touched by nothing
    // above (full blocks end below it, a partly filled one excludes it), so this needs no ordering with the loops above.
    if (len)
        for (int r = blockIdx.x * blockDim.x + threadIdx.x; r < ps.R; r += gridDim.x * blockDim.x)
            append_row(ps, r, len, done, status);
}

// item = (rewritten slot m, pool q): all heads of the live positions of one block
__global__ void __launch_bounds__(256) paged_copy_kernel(const PagedState ps, const PagedPools pools,
                                                         const int32_t* n_moves) {
    chain_begin();
    const int n = *n_moves;
    if (n <= 0) return;
    const CopyOrder* orders = orders_of(ps);
    const int n_pools = 2 * pools.n_layers;
    const int64_t head_bytes = (int64_t)ps.block_len * pools.pos_bytes, blk_bytes = head_bytes * pools.H;
    const int64_t total = (int64_t)n * n_pools;
    for (int64_t w = blockIdx.x; w < total; w += gridDim.x) {
        const int m = (int)(w / n_pools), q = (int)(w - (int64_t)m * n_pools);
        const CopyOrder o = orders[m];
        if (o.positions <= 0) continue;
        char* pool = (q & 1) ? pools.v[q >> 1] : pools.k[q >> 1];
        const uint4* src = reinterpret_cast<const uint4*>(pool + (int64_t)o.src_blk * blk_bytes);
        uint4* dst = reinterpret_cast<uint4*>(pool + (int64_t)o.dst_blk * blk_bytes);
        const int per_head = o.positions * pools.pos_bytes / 16, stride = (int)(head_bytes / 16);
        const int n_el = per_head * pools.H;
        // Four loads in flight per thread, then their stores: source and destination lie in one pool, so a plain
        // copy loop would wait for every load before it may issue the next store (one trip to memory per element;
        // measured on 512 rows with 32 layers: the three kernels of a reindex 31.2 -> 25.7 us, eight loads 27.1 us).
        constexpr int kBatch = 4;
        for (int e0 = threadIdx.x; e0 < n_el; e0 += kBatch * blockDim.x) {
            uint4 v[kBatch];
            int64_t at[kBatch];
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const int e = e0 + u * (int)blockDim.x;
                at[u] = -1;
                if (e < n_el) {
                    const int h = e / per_head, x = e - h * per_head;
                    at[u] = (int64_t)h * stride + x;
                    v[u] = src[at[u]];
                }
            }
#pragma unroll
            for (int u = 0; u < kBatch; ++u)
                if (at[u] >= 0) dst[at[u]] = v[u];
        }
    }
}

}  // namespace

size_t paged_free_list_words(int n_blocks, int R) {  // the free list, then one 12-byte copy order per row
    return (size_t)n_blocks + 3 * (size_t)R;
}

cudaError_t launch_paged_init(const PagedState& ps, const int32_t* prompt_len_dev, int G, int share_prompt,
                              int32_t* status, cudaStream_t stream) {
    paged_init_kernel<<<1, 1024, 0, stream>>>(ps, prompt_len_dev, G, share_prompt, status);
    return cudaGetLastError();
}

cudaError_t launch_paged_append(const PagedState& ps, const int32_t* len, const uint8_t* done, int32_t* status,
                                cudaStream_t stream) {
    return launch_chained(paged_append_kernel, dim3((unsigned)((ps.R + 255) / 256)), dim3(256), 0, stream, ps, len, done,
                          status);
}

cudaError_t launch_paged_reindex(const PagedState& ps, const PagedPools& pools, const MoveSource* sources,
                                 const int32_t* dst_rows, const int32_t* n_sources, const int32_t* n_moves,
                                 const int32_t* len, const uint8_t* done, int32_t* status, cudaStream_t stream) {
    cudaError_t e = launch_chained(paged_release_kernel, dim3(kSMs), dim3(256), 0, stream, ps, dst_rows, n_moves);
    if (e != cudaSuccess) return e;
    // a warp per source; there are at most R / 2 of them (each has at least one destination besides itself)
    e = launch_chained(paged_acquire_kernel, dim3((unsigned)((ps.R / 2 + 7) / 8 + 1)), dim3(256), 0, stream, ps, sources,
                       dst_rows, n_sources, len, done, status);
    if (e != cudaSuccess) return e;
    // items = rewritten slots x pools; about an eighth of the rows are rewritten in a step with resampling
    int64_t ctas = (int64_t)(ps.R / 8 + 1) * (2 * pools.n_layers);
    ctas = ctas < kSMs ? kSMs : (ctas > kSMs * 16 ? kSMs * 16 : ctas);
    return launch_chained(paged_copy_kernel, dim3((unsigned)ctas), dim3(256), 0, stream, ps, pools, n_moves);
}

}  // namespace psmc
