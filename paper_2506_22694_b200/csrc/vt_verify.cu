// Greedy verification of drafted blocks (Experiments section: the target decodes greedily and a draft
// token counts only when it equals the target's token; the accept loop of Algorithm 2) and the token
// count behind the block efficiency tau.  Pure id comparison: one warp walks one sequence's tree.
#include "vt_common.cuh"

#include <climits>

namespace vt {
namespace {

constexpr int kWarpsPerCta = 8;

__global__ void __launch_bounds__(kWarpsPerCta * 32)
k_verify_greedy(const int32_t* __restrict__ token, const int32_t* __restrict__ parent,
                const int32_t* __restrict__ target, int32_t S, int32_t N, int32_t* __restrict__ n_accept,
                int32_t* __restrict__ path, int32_t* __restrict__ emitted, unsigned long long* tokens_total) {
    const int lane = threadIdx.x & 31;
    const int64_t s = (int64_t)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
    if (s >= S) return;                                            // whole warps leave together
    const int32_t* tok = token + s * N;
    const int32_t* par = parent ? parent + s * N : nullptr;
    const int32_t* tgt = target + s * ((int64_t)N + 1);
    int32_t* my_path = path ? path + s * N : nullptr;
    int32_t* my_emit = emitted ? emitted + s * ((int64_t)N + 1) : nullptr;
    if (my_path) for (int i = lane; i < N; i += 32) my_path[i] = -1;
    if (my_emit) for (int i = lane; i <= N; i += 32) my_emit[i] = -1;
    __syncwarp();
    int cur = -1, n = 0;
    for (;;) {                                                     // every quantity steering the loops is warp-uniform
        const int32_t want = tgt[cur + 1];
        int next = INT_MAX;
        for (int base = cur + 1; base < N; base += 32) {           // children have larger indices than their parent
            const int i = base + lane;
            bool hit = false;
            if (i < N) {
                const int32_t p = par ? par[i] : i - 1;
                hit = (p == cur) & (tok[i] == want);
            }
            const unsigned m = __ballot_sync(0xffffffffu, hit);
            if (m) { next = base + __ffs(m) - 1; break; }          // lowest index among equal siblings
        }
        if (next == INT_MAX) break;
        if (lane == 0) {
            if (my_path) my_path[n] = next;
            if (my_emit) my_emit[n] = tok[next];
        }
        ++n;
        cur = next;
    }
    if (lane == 0) {
        if (my_emit) my_emit[n] = tgt[cur + 1];                    // the target's own token closes the block
        n_accept[s] = n;
        if (tokens_total) atomicAdd(tokens_total, (unsigned long long)(n + 1));
    }
}

}  // namespace

cudaError_t launch_verify_greedy(const int32_t* token, const int32_t* parent, const int32_t* target, int32_t S,
                                 int32_t N, int32_t* n_accept, int32_t* path, int32_t* emitted,
                                 unsigned long long* tokens_total, cudaStream_t st) {
    if (S == 0) return cudaSuccess;
    const unsigned grid = (unsigned)((S + kWarpsPerCta - 1) / kWarpsPerCta);
    k_verify_greedy<<<grid, kWarpsPerCta * 32, 0, st>>>(token, parent, target, S, N, n_accept, path, emitted,
                                                        tokens_total);
    count_launch();
    return cudaGetLastError();
}

}  // namespace vt
