// Draft-tree expansion as a block-wide device function, shared by the stand-alone kernel and by the
// head kernel that runs it right after its merge (Settings: tree construction following EAGLE-2).
#pragma once
#include "vt_common.cuh"

namespace vt {
namespace {

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

// One depth of the expansion by the `nthreads` threads `tid` of a CTA that all call it; s_key holds
// B * topk keys.  Contains two CTA barriers.
__device__ __forceinline__ void tree_expand_block(const TreeArgs& t, const int32_t* __restrict__ cand_ids,
                                                  const float* __restrict__ cand_lp, int32_t B, int32_t topk,
                                                  int32_t ld, int32_t col0, unsigned long long* s_key, int tid,
                                                  int nthreads) {
    const int n_new = B * topk;
    for (int i = tid; i < n_new; i += nthreads) {
        const int b = i / topk, j = i - b * topk;
        int32_t par = t.frontier ? t.frontier[b] : -1;
        if (par < -1 || par >= t.pool_base) par = -1;                   // memory safety; callers pass earlier nodes
        const float base = par < 0 ? 0.0f : t.pool_score[par];         // earlier depth: not written by this launch
        const float lp = cand_lp[(int64_t)b * ld + col0 + j];
        const float step = (lp != lp) ? lp : fminf(lp, 0.0f);          // a log-probability is never positive
        const float s = base + step;
        const int node = t.pool_base + i;
        t.pool_token[node] = cand_ids[(int64_t)b * ld + col0 + j];
        t.pool_parent[node] = par;
        t.pool_score[node] = s;
        s_key[i] = node_key(s, i);
    }
    __syncthreads();
    for (int i = tid; i < n_new; i += nthreads) {
        const int r = rank_of(s_key, n_new, s_key[i]);
        if (r < t.n_front) t.next_frontier[r] = t.pool_base + i;
    }
}

}  // namespace
}  // namespace vt
