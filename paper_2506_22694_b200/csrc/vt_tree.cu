// Draft-tree construction around the head (Settings: "draft trees construction ... following EAGLE-2",
// depth 3 / top-K 8 / 32 draft tokens, 60 in the depth ablation).  Two on-chip selections over at most
// a few thousand values: the frontier of the next depth, and the final rerank of the node pool.
// Scores are cumulative log-probabilities in fp32; ties go to the lower node index; NaN ranks last.
#include "vt_common.cuh"

namespace vt {
namespace {

constexpr int kTreeThreads = 1024;
constexpr int kTreeMax = 4096;                       // nodes one call ranks (VT_TREE_MAX_NODES)

__device__ __forceinline__ uint32_t score_ord(float s) {
    if (s != s) s = __int_as_float(0xff800000);      // NaN ranks with -inf
    if (s == 0.0f) s = 0.0f;                         // one zero
    const uint32_t u = __float_as_uint(s);
    return u ^ ((u >> 31) ? 0xffffffffu : 0x80000000u);
}

__device__ __forceinline__ unsigned long long node_key(float s, int i) {
    return ((unsigned long long)score_ord(s) << 32) | (uint32_t)~(uint32_t)i;     // greater key = preferred
}

// rank of keys[i] among keys[0..n): number of strictly greater keys (keys are distinct)
__device__ __forceinline__ int rank_of(const unsigned long long* keys, int n, unsigned long long mine) {
    int r = 0;
    for (int j = 0; j < n; ++j) r += keys[j] > mine;  // all lanes read the same word: a broadcast
    return r;
}

__global__ void __launch_bounds__(kTreeThreads, 1)
k_tree_expand(const int32_t* __restrict__ cand_ids, const float* __restrict__ cand_lp, int32_t B, int32_t topk,
              int32_t ld, int32_t col0, const int32_t* __restrict__ frontier, int32_t* __restrict__ pool_token,
              int32_t* __restrict__ pool_parent, float* pool_score, int32_t pool_base, int32_t n_front,
              int32_t* __restrict__ next_frontier) {
    __shared__ unsigned long long s_key[kTreeMax];
    const int n_new = B * topk;
    for (int i = threadIdx.x; i < n_new; i += kTreeThreads) {
        const int b = i / topk, j = i - b * topk;
        int32_t par = frontier ? frontier[b] : -1;
        if (par < -1 || par >= pool_base) par = -1;                     // memory safety; callers pass earlier nodes
        const float base = par < 0 ? 0.0f : pool_score[par];           // earlier depth: not written by this launch
        const float lp = cand_lp[(int64_t)b * ld + col0 + j];
        const float step = (lp != lp) ? lp : fminf(lp, 0.0f);          // a log-probability is never positive
        const float s = base + step;
        const int node = pool_base + i;
        pool_token[node] = cand_ids[(int64_t)b * ld + col0 + j];
        pool_parent[node] = par;
        pool_score[node] = s;
        s_key[i] = node_key(s, i);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n_new; i += kTreeThreads) {
        const int r = rank_of(s_key, n_new, s_key[i]);
        if (r < n_front) next_frontier[r] = pool_base + i;
    }
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
                               int32_t col0, const int32_t* frontier, int32_t* pool_token, int32_t* pool_parent,
                               float* pool_score, int32_t pool_base, int32_t n_front, int32_t* next_frontier,
                               cudaStream_t st) {
    k_tree_expand<<<1, kTreeThreads, 0, st>>>(cand_ids, cand_lp, B, topk, ld, col0, frontier, pool_token,
                                              pool_parent, pool_score, pool_base, n_front, next_frontier);
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
