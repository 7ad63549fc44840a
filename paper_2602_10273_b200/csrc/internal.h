// Host-side declarations shared by the translation units of libpsmc.so.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/psmc.h"

namespace psmc {

// Launch with programmatic stream serialisation: the kernel may be scheduled (and run up to its chain_begin())
// while the previous kernel of the stream drains, which hides launch latency between the kernels of a step.
// Every kernel launched this way calls chain_begin() before it touches global memory, and every grid of the
// step fits the GPU in one wave, so early CTAs never keep a predecessor's CTAs from being scheduled.
// Opt a kernel in to `bytes` of dynamic shared memory on the current device (the attribute is per function and per
// device); remembered per (kernel, device), so the runtime is asked once each.
cudaError_t allow_dynamic_smem(const void* kernel, int bytes);

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                  Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

constexpr int kMaxParticles = 1024;  // one CTA per group in the weight/resample kernel
constexpr int kSMs = 148;            // B200

// ---------------------------------------------------------------- logit pass (Eq. 7, Corollary 1)
struct LogitsStreamArgs {
    const void* logits;
    int dt;          // psmc_dtype
    int R, V;
    int64_t ld;
    double beta;
    const uint8_t* done;   // may be NULL
    void* scratch;         // span triples, logits_pass_scratch_bytes(R, V)
    int32_t* zero_words;   // optional: two consecutive words the kernel clears before anything else (may be NULL)
    int32_t* status;       // sticky status word for a bounded wait that ran out (may be NULL)
};
struct LogitsGeometry {    // how a [R, V] block is cut up; a pure function of the arguments
    int span, n_spans, mode, vec;
    float bf;             // (float)beta
};
int logits_pass_span(int R, int V);               // logits per warp task
size_t logits_pass_scratch_bytes(int R, int V);
LogitsGeometry logits_geometry(const void* logits, int dt, int R, int V, int64_t ld, double beta);
cudaError_t launch_logits_stream(const LogitsStreamArgs& a, cudaStream_t stream);

// ---------------------------------------------------------------- weights, ESS, resampling
struct MoveSource {      // one surviving particle with surplus offspring
    int32_t src_row;     // row to read
    int32_t len;         // positions [0, len) to copy
    int32_t dst_begin;   // first entry of its destinations in the destination list
    int32_t n_dst;       // how many rows receive it
};
struct WeightsArgs {
    int G, N, R, t, eos;
    int resampler;  // psmc_resampler
    double alpha_t, beta, delta, kappa;
    uint64_t seed;
    // the logit block of this step and the span triples the streaming kernel left
    const void* logits;
    int dt, V;
    int64_t ld;
    const void* scratch;
    // per-row results of the finish (written here; zero for finished rows)
    double* logp;
    double* loginc;
    // particle state, updated in place
    double* logW;
    double* S;
    const uint8_t* done;  // finished flags as the step finds them: read only, by any CTA at any time during the step
    uint8_t* done_out;    // finished flags after the step (another array: a group may close while other CTAs still look
                          // at the flags of its rows)
    int32_t* len;
    // per-step results
    int32_t* tok;       // [R] token of each slot this step (EOS for finished rows)
    int32_t* last_tok;  // [R] after the map
    int32_t* anc;
    int32_t* map;
    int32_t* resampled; // [G]
    double* ess;        // [G]
    double* logZ;       // [G]
    int32_t* hist_tok;  // row t-1 of [T_max][R]
    int32_t* hist_map;
    // move records for the cache reindex
    MoveSource* sources;
    int32_t* dst_rows;
    int32_t* n_sources;  // [1]
    int32_t* n_moves;    // [1]
    int32_t* status;
};
cudaError_t launch_weights_resample(const WeightsArgs& a, cudaStream_t stream);

// The logit pass and the per-group update as one kernel (step_fused.cu): possible for groups of up to 32 particles
// whose logit rows start on 16-byte boundaries.  shared_triples: step_fused_scratch_bytes() of device memory, contents
// irrelevant; row_arrivals [R] and group_arrivals [G] are zero between launches (the kernel leaves them so).
bool step_can_fuse(const LogitsStreamArgs& la, int N);
size_t step_fused_scratch_bytes();
cudaError_t launch_step_fused(const LogitsStreamArgs& la, const WeightsArgs& wa, void* shared_triples,
                              int32_t* row_arrivals, int32_t* group_arrivals, cudaStream_t stream);

// The step with the proposal restricted to the top_k tokens of each row, or to the nucleus of share top_p (exactly one
// of the two > 0): one CTA per row for the logit pass, then the per-group update.  set_size: [R].
cudaError_t launch_rows_weights(const WeightsArgs& wa, cudaStream_t stream);  // group updates from rows already in memory
cudaError_t launch_step_masked(const LogitsStreamArgs& la, const WeightsArgs& wa, int top_k, double top_p,
                               int32_t* set_size, cudaStream_t stream);

// ---------------------------------------------------------------- the step with the vocabulary split over ranks
struct ShardLocateArgs {
    const double* all_triples;  // [P][R][3]
    int P, rank, N, t, v0;
    int tile_width;             // 0: rank `rank` holds columns from v0 on.  > 0: the parts are vocabulary tiles of this
                                // width fed one after the other, and row r of the logits given holds the columns of
                                // the tile that owns row r (its own tile for every row)
    double alpha_t;
    uint64_t seed;
    psmc_shard_pick* picks_out;  // [R]
};
// la describes the local columns (V = their number); its scratch holds the span triples of the streaming kernel
cudaError_t launch_shard_triples(const LogitsStreamArgs& la, double* triples_out, cudaStream_t stream);
cudaError_t launch_shard_locate(const LogitsStreamArgs& la, const ShardLocateArgs& sa, cudaStream_t stream);
// a.logits / a.scratch are not used: the row results come from the gathered triples and picks.
// picks_per_row: all_picks is [R] (row r's pick whoever its owner is) instead of [P][R].
cudaError_t launch_shard_weights(const WeightsArgs& a, const double* all_triples, const psmc_shard_pick* all_picks, int P,
                                 cudaStream_t stream, bool picks_per_row = false);
// need_out[r] = first column of the part (tile) that holds row r's target mass, -1 for a finished or unusable row
cudaError_t launch_shard_owner_columns(const double* all_triples, int P, int R, int N, int t, double beta, uint64_t seed,
                                       const uint8_t* done, int tile_width, int32_t* need_out, cudaStream_t stream);

// ---------------------------------------------------------------- KV reindex (Appendix C)
constexpr int kMaxKvPtrs = 128;  // K and V pointers per launch (64 layers); more layers take more launches
struct KvLaunch {
    char* src[kMaxKvPtrs];
    char* dst[kMaxKvPtrs];
    int n_ptrs;
    int H;
    int64_t row_bytes_stride, head_bytes_stride;  // bytes
    int64_t dst_row_bytes_stride, dst_head_bytes_stride;
    int pos_bytes;   // head_dim * sizeof(elem)
    int max_len;
    const MoveSource* sources;
    const int32_t* dst_rows;
    const int32_t* n_sources;
    int32_t* status;
    const int32_t* skip_pos;  // [G] positions at the start of every row of group g that are not copied, or NULL
    int N;                    // particles per group (rows per entry of skip_pos)
    int32_t* work;   // [2] unit queue of the copy kernels: next unit, CTAs that have left; both zero between launches
    int bulk_ok;     // 16-byte alignment holds everywhere
};
cudaError_t launch_reindex_kv(const KvLaunch& k, cudaStream_t stream);
int reindex_unit_parts();  // work units per (source row, tensor, head): rows * pointers * heads * this must stay below 2^31
// turn an arbitrary gather vector into move records (and check in-place hazards)
cudaError_t launch_build_moves(const int32_t* idx, int R, int max_len, int in_place, MoveSource* sources,
                               int32_t* dst_rows, int32_t* n_sources, int32_t* n_moves, int32_t* status,
                               cudaStream_t stream);

// ---------------------------------------------------------------- paged KV cache (block table, copy on write)
struct PagedState {
    int32_t* table;      // [R][max_blocks]
    int32_t* refc;       // [n_blocks]
    int32_t* free_list;  // [n_blocks] stack; entries [0, *free_top) are free
    int32_t* free_top;   // [1]
    int n_blocks, block_len, max_blocks, R, N;
};
struct PagedPools {
    char* k[kMaxKvPtrs / 2];
    char* v[kMaxKvPtrs / 2];
    int n_layers, H;
    int pos_bytes;       // head_dim * sizeof(elem)
};
size_t paged_free_list_words(int n_blocks, int R);  // words to allocate for PagedState::free_list
cudaError_t launch_paged_init(const PagedState& ps, const int32_t* prompt_len_dev, int G, int share_prompt,
                              int32_t* status, cudaStream_t stream);
cudaError_t launch_paged_append(const PagedState& ps, const int32_t* len, const uint8_t* done, int32_t* status,
                                cudaStream_t stream);
// len / done: NULL, or the rows' lengths and finished flags after the step: every live row then also gets the block
// its next position needs
cudaError_t launch_paged_reindex(const PagedState& ps, const PagedPools& pools, const MoveSource* sources,
                                 const int32_t* dst_rows, const int32_t* n_sources, const int32_t* n_moves,
                                 const int32_t* len, const uint8_t* done, int32_t* status, cudaStream_t stream);

// ---------------------------------------------------------------- final draw and back-trace
struct SelectArgs {
    int G, N, R, t, T_max, eos;
    uint64_t seed;
    const double* logW;
    const int32_t* hist_tok;
    const int32_t* hist_map;
    int32_t* out_tokens;
    int32_t* out_len;
    int32_t* out_index;
};
cudaError_t launch_select(const SelectArgs& a, cudaStream_t stream);

}  // namespace psmc
