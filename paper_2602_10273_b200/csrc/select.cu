// Output step of Algorithm 1: per group draw I ~ Categorical(W) and return the token string of
// particle I.  Prefixes are not copied at resampling time; each step logs the tokens drawn and the
// slot map applied, and the string is recovered here by walking that log backwards:
//   cur = I;  for t = T..1:  cur = map_t[cur];  y_t = tok_t[cur].
// One CTA per group.  The log rows of a batch of steps are staged in shared memory by all threads,
// then one thread walks the batch, so the dependent chain never waits on global memory.
#include "common.cuh"
#include "internal.h"

namespace psmc {
namespace {

constexpr int kSelThreads = 256;
constexpr int kStageInts = 4096;  // per array: steps_per_batch * N <= kStageInts

__global__ void __launch_bounds__(kSelThreads) select_kernel(const SelectArgs a) {
    __shared__ double sh_red[33];
    __shared__ double sh_w[kMaxParticles];
    __shared__ int sh_map[kStageInts];
    __shared__ int sh_tok[kStageInts];
    __shared__ int sh_cur, sh_first_eos;

    const int g = blockIdx.x, N = a.N, tid = threadIdx.x;
    const double* lw = a.logW + (size_t)g * N;

    // weights relative to the largest, then the inverse CDF over slots in order
    double mx = -INFINITY;
    for (int i = tid; i < N; i += blockDim.x) mx = fmax(mx, lw[i]);
    mx = block_max(mx, sh_red, (int)(blockDim.x >> 5));
    for (int i = tid; i < N; i += blockDim.x) sh_w[i] = exp(lw[i] - mx);
    __syncthreads();
    if (tid == 0) {
        double s1 = 0.0;
        for (int i = 0; i < N; ++i) s1 += sh_w[i];
        const double U = hash_uniform(hash5(a.seed, kStreamSelect, (uint64_t)g, 0, 0));
        const double target = U * s1;
        double cum = 0.0;
        int I = N - 1;
        for (int i = 0; i < N; ++i) {
            cum += sh_w[i];
            if (cum >= target) {
                I = i;
                break;
            }
        }
        sh_cur = I;
        sh_first_eos = -1;
        if (a.out_index) a.out_index[g] = I;
    }
    __syncthreads();

    // walk the log backwards in batches of `bs` steps
    const int bs = kStageInts / N;
    for (int t_hi = a.t; t_hi >= 1; t_hi -= bs) {
        const int t_lo = max(1, t_hi - bs + 1);  // batch covers steps t_lo..t_hi
        const int steps = t_hi - t_lo + 1;
        for (int e = tid; e < steps * N; e += blockDim.x) {
            const int s = e / N, i = e - s * N;
            const size_t off = (size_t)(t_lo - 1 + s) * a.R + (size_t)g * N + i;
            sh_map[e] = a.hist_map[off];
            sh_tok[e] = a.hist_tok[off];
        }
        __syncthreads();
        if (tid == 0) {
            int cur = sh_cur, first_eos = sh_first_eos;
            for (int s = steps - 1; s >= 0; --s) {
                cur = sh_map[s * N + cur];
                const int tok = sh_tok[s * N + cur];
                sh_tok[s * N] = tok;  // slot 0 of the step's row is reused as the output cell
                if (tok == a.eos) first_eos = t_lo + s;
            }
            sh_cur = cur;
            sh_first_eos = first_eos;
        }
        __syncthreads();
        if (a.out_tokens)
            for (int s = tid; s < steps; s += blockDim.x)
                a.out_tokens[(size_t)g * a.T_max + (t_lo - 1 + s)] = sh_tok[s * N];
        __syncthreads();
    }
    if (a.out_tokens)
        for (int t = a.t + tid; t < a.T_max; t += blockDim.x) a.out_tokens[(size_t)g * a.T_max + t] = -1;
    if (tid == 0 && a.out_len) a.out_len[g] = sh_first_eos > 0 ? sh_first_eos : a.t;
}

}  // namespace

cudaError_t launch_select(const SelectArgs& a, cudaStream_t stream) {
    select_kernel<<<a.G, kSelThreads, 0, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace psmc
