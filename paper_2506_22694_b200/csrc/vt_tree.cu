// Draft-tree construction around the head (Section 4.1, Settings: the EAGLE-2 tree procedure with
// depth 3 / top-K 8 / 32 draft tokens; Table 4: 60 draft tokens in the depth ablation).  Two on-chip selections over at most
// a few thousand values: the frontier of the next depth, and the final rerank of the node pool.
// Scores are cumulative log-probabilities in fp32; ties go to the lower node index; NaN ranks last.
#include "vt_common.cuh"
#include "vt_tree_common.cuh"

namespace vt {
namespace {

constexpr int kTreeThreads = 1024;
constexpr int kTreeMax = 4096;                       // nodes one call ranks (VT_TREE_MAX_NODES)

__global__ void __launch_bounds__(kTreeThreads, 1)
k_tree_expand(const int32_t* __restrict__ cand_ids, const float* __restrict__ cand_lp, int32_t B, int32_t topk,
              int32_t ld, int32_t col0, const TreeArgs t) {
    __shared__ unsigned long long s_key[kTreeMax];
    tree_expand_block(t, cand_ids, cand_lp, B, topk, ld, col0, s_key, (int)threadIdx.x, kTreeThreads);
}

__global__ void __launch_bounds__(kTreeThreads, 1)
k_tree_rerank(const int32_t* __restrict__ pool_token, const int32_t* __restrict__ pool_parent,
              const float* __restrict__ pool_score, int32_t n, int32_t budget, int32_t* __restrict__ out_nodes,
              int32_t* __restrict__ out_token, int32_t* __restrict__ out_parent) {
    __shared__ unsigned long long s_key[kTreeMax];
    __shared__ uint32_t s_sel[kTreeMax / 32];        // bit i: node i is kept
    __shared__ int s_before[kTreeMax / 32];          // kept nodes in earlier words
    for (int i = threadIdx.x; i < n; i += kTreeThreads) s_key[i] = node_key(pool_score[i], i);
    for (int w = threadIdx.x; w < kTreeMax / 32; w += kTreeThreads) s_sel[w] = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += kTreeThreads)
        if (rank_of(s_key, n, s_key[i]) < budget) atomicOr(&s_sel[i >> 5], 1u << (i & 31));
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int w = 0; w < kTreeMax / 32; ++w) { s_before[w] = run; run += __popc(s_sel[w]); }
    }
    __syncthreads();
    const int m = min(budget, n);
    for (int i = threadIdx.x; i < n; i += kTreeThreads) {
        const uint32_t bit = 1u << (i & 31);
        if (!(s_sel[i >> 5] & bit)) continue;
        const int pos = s_before[i >> 5] + __popc(s_sel[i >> 5] & (bit - 1));
        const int32_t par = pool_parent[i];
        int32_t ppos = -1;
        if (par >= 0) {
            const bool ok = par < n && (s_sel[par >> 5] >> (par & 31) & 1u);
            ppos = ok ? s_before[par >> 5] + __popc(s_sel[par >> 5] & ((1u << (par & 31)) - 1)) : -2;
        }
        out_nodes[pos] = i;
        out_token[pos] = pool_token[i];
        out_parent[pos] = ppos;
    }
    for (int k = m + threadIdx.x; k < budget; k += kTreeThreads) {
        out_nodes[k] = -1;
        out_token[k] = -1;
        out_parent[k] = -1;
    }
}

}  // namespace

int tree_max_nodes() { return kTreeMax; }

cudaError_t launch_tree_expand(const int32_t* cand_ids, const float* cand_lp, int32_t B, int32_t topk, int32_t ld,
                               int32_t col0, const TreeArgs& t, cudaStream_t st) {
    k_tree_expand<<<1, kTreeThreads, 0, st>>>(cand_ids, cand_lp, B, topk, ld, col0, t);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_tree_rerank(const int32_t* pool_token, const int32_t* pool_parent, const float* pool_score,
                               int32_t n, int32_t budget, int32_t* out_nodes, int32_t* out_token,
                               int32_t* out_parent, cudaStream_t st) {
    k_tree_rerank<<<1, kTreeThreads, 0, st>>>(pool_token, pool_parent, pool_score, n, budget, out_nodes, out_token,
                                              out_parent);
    count_launch();
    return cudaGetLastError();
}

}  // namespace vt
