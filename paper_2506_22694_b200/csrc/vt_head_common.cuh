// Pieces shared by the two head kernels (streaming and dense): ordering helpers, the per-CTA record
// layout and the cross-CTA merge that turns the records into out_ids / out_logprobs.
#pragma once
#include <math_constants.h>

#include "vt_common.cuh"

namespace vt {
namespace {

constexpr int kMaxGrid = 160;                    // merge: each lane owns at most kMaxOwn CTA records
constexpr int kMaxOwn = kMaxGrid / 32;
constexpr int kMergeDepth = 4;                   // list entries per CTA staged on chip by the merge
constexpr int kSelCap = 128;                     // entries the merge's direct selection can rank
constexpr int kMergeStageWords = 2 * kMergeDepth * kMaxGrid + 2 * kSelCap + 64;   // staging floats per merging warp

__host__ __device__ inline int rec_fields(int topk) { return 5 + 2 * topk; }

__device__ __forceinline__ bool better(float v, int j, float bv, int bj) {
    return v > bv || (v == bv && j < bj);
}

// (m, s) <- (m, s) (+) (m2, s2) for running max / sum of exponentials
__device__ __forceinline__ void lse_merge(float& m, float& s, float m2, float s2) {
    const float M = fmaxf(m, m2);
    if (M == -CUDART_INF_F) { m = M; s = 0.f; return; }
    s = s * __expf(m - M) + s2 * __expf(m2 - M);
    m = M;
}


// Order-preserving map of a float onto unsigned integers (and back); no NaN ever reaches it.
__device__ __forceinline__ unsigned f2ord(float f) {
    const unsigned u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float ord2f(unsigned k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// (value, index) as one unsigned 64-bit key: larger key = better candidate (higher value, then lower
// index).  Comparing keys needs no data-dependent branch; per-lane branches inside a warp cost far
// more than the arithmetic they skip.
__device__ __forceinline__ unsigned long long key64(float v, int j) {
    return ((unsigned long long)f2ord(v) << 32) | (unsigned)(~j);
}
__device__ __forceinline__ float key_val(unsigned long long k) { return ord2f((unsigned)(k >> 32)); }
__device__ __forceinline__ int key_idx(unsigned long long k) { return (int)~(unsigned)k; }

// Records: one word per (hidden row b, field f, CTA c) at recs[(b * rec_fields(topk) + f) * kMaxGrid + c],
// CTA index fastest so that the merging warp reads every field with coalesced loads.
// Fields: 0 m, 1 s, 2 Gumbel score, 3 Gumbel j, 4 Gumbel z, 5+r value of list entry r, 5+topk+r its index.
__device__ __forceinline__ size_t rec_at(int b, int f, int topk) {
    return ((size_t)b * rec_fields(topk) + f) * kMaxGrid;
}

// Last CTA: merge all CTA records of hidden row b in CTA order (one warp per row), remap through
// `map`, write the outputs.  All loads of a phase are issued before the first use, so the merge
// costs a couple of L2 round trips.  `stage` is idle shared memory for the heads of the lists.
struct MergeOut {
    const int32_t* map;
    int32_t* out_ids;
    float* out_logprobs;
    float* dbg_lse;
    int topk;
    int sampled;       // uniforms were given: column 0 is the Gumbel-max draw
};
__device__ __noinline__ void merge_records(const int32_t* map, int32_t* out_ids, float* out_logprobs, float* dbg_lse,
                                           int topk, int sampled, Ctrl* ctrl, const float* recs, int b, bool row_ok,
                                           int G, float* stv) {
    const MergeOut a{map, out_ids, out_logprobs, dbg_lse, topk, sampled};
    const int lane = threadIdx.x & 31;
    const int* irecs = reinterpret_cast<const int*>(recs);
    const int depth = min(topk, kMergeDepth);
    float hm[kMaxOwn], hs[kMaxOwn], hgs[kMaxOwn], hgz[kMaxOwn];
    int hgj[kMaxOwn];
    float ev[kMergeDepth][kMaxOwn];
    int ej[kMergeDepth][kMaxOwn];
#pragma unroll
    for (int o = 0; o < kMaxOwn; ++o) {
        const int c = lane + 32 * o;
        const bool on = c < G;
        hm[o] = on ? ld_cg_f32(recs + rec_at(b, 0, topk) + c) : -CUDART_INF_F;
        hs[o] = on ? ld_cg_f32(recs + rec_at(b, 1, topk) + c) : 0.f;
        hgs[o] = on ? ld_cg_f32(recs + rec_at(b, 2, topk) + c) : -CUDART_INF_F;
        hgj[o] = on ? ld_cg_s32(irecs + rec_at(b, 3, topk) + c) : -1;
        hgz[o] = on ? ld_cg_f32(recs + rec_at(b, 4, topk) + c) : 0.f;
#pragma unroll
        for (int r = 0; r < kMergeDepth; ++r) {
            const bool on2 = on && r < depth;
            ev[r][o] = on2 ? ld_cg_f32(recs + rec_at(b, 5 + r, topk) + c) : -CUDART_INF_F;
            ej[r][o] = on2 ? ld_cg_s32(irecs + rec_at(b, 5 + topk + r, topk) + c) : -1;
        }
    }
    float M = -CUDART_INF_F, Ssum = 0.f, GS = -CUDART_INF_F, GZ = 0.f;
    int GJ = -1;
#pragma unroll
    for (int o = 0; o < kMaxOwn; ++o) {
        lse_merge(M, Ssum, hm[o], hs[o]);
        if (hgj[o] >= 0 && (GJ < 0 || better(hgs[o], hgj[o], GS, GJ))) { GS = hgs[o]; GJ = hgj[o]; GZ = hgz[o]; }
    }
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, M, o), s2 = __shfl_xor_sync(0xffffffffu, Ssum, o);
        lse_merge(M, Ssum, m2, s2);
        const float gs2 = __shfl_xor_sync(0xffffffffu, GS, o), gz2 = __shfl_xor_sync(0xffffffffu, GZ, o);
        const int gj2 = __shfl_xor_sync(0xffffffffu, GJ, o);
        if (gj2 >= 0 && (GJ < 0 || better(gs2, gj2, GS, GJ))) { GS = gs2; GJ = gj2; GZ = gz2; }
    }
    const float lse = M + logf(Ssum);
    float res_v[2] = {0.f, 0.f};
    int res_j[2] = {-1, -1};
    bool done = false;
    if (topk <= 32) {
        // Direct selection.  tau = the topk-th largest of the 32 lanes' best list heads is a lower
        // bound of the topk-th best entry overall, so only staged entries >= tau can matter: a few
        // dozen at most.  They are compacted into shared memory and every one finds its output
        // position as its rank -- no sequential rounds.  Falls back to the rounds below when a list
        // might hold qualifying entries beyond the staged ones, or when too many qualify.
        unsigned lh = 0u;
#pragma unroll
        for (int o = 0; o < kMaxOwn; ++o) {
            const bool live = (lane + 32 * o < G) && ej[0][o] >= 0;
            const unsigned h = live ? f2ord(ev[0][o]) : 0u;
            lh = h > lh ? h : lh;
        }
        int rk = 0;
#pragma unroll
        for (int sl = 0; sl < 32; ++sl) {
            const unsigned oh = __shfl_sync(0xffffffffu, lh, sl);
            rk += (oh > lh || (oh == lh && sl < lane)) ? 1 : 0;
        }
        const unsigned at = __ballot_sync(0xffffffffu, rk == topk - 1);
        const unsigned tau = __shfl_sync(0xffffffffu, lh, __ffs(at) - 1);
        unsigned long long* sel = reinterpret_cast<unsigned long long*>(stv + 2 * kMergeDepth * kMaxGrid);
        unsigned long long* outk = sel + kSelCap;
        outk[lane] = 0ull;
        int n = 0;
        bool deep = false;
#pragma unroll
        for (int r = 0; r < kMergeDepth; ++r)
#pragma unroll
            for (int o = 0; o < kMaxOwn; ++o) {
                const bool in = (lane + 32 * o < G) && r < depth && ej[r][o] >= 0 && f2ord(ev[r][o]) >= tau;
                const unsigned bm = __ballot_sync(0xffffffffu, in);
                if (in) {
                    const int pos = n + __popc(bm & lanemask_lt());
                    if (pos < kSelCap) sel[pos] = key64(ev[r][o], ej[r][o]);
                }
                n += __popc(bm);
                deep = deep || (in && r == depth - 1 && depth < topk);
            }
        if (n <= kSelCap && !__any_sync(0xffffffffu, deep)) {
            __syncwarp();
            unsigned long long mine[kSelCap / 32];
            int rk4[kSelCap / 32];
#pragma unroll
            for (int i = 0; i < kSelCap / 32; ++i) {
                mine[i] = (lane + 32 * i < n) ? sel[lane + 32 * i] : 0ull;
                rk4[i] = 0;
            }
            for (int e = 0; e < n; ++e) {
                const unsigned long long k = sel[e];
#pragma unroll
                for (int i = 0; i < kSelCap / 32; ++i) rk4[i] += (k > mine[i]) ? 1 : 0;
            }
#pragma unroll
            for (int i = 0; i < kSelCap / 32; ++i)
                if (lane + 32 * i < n && rk4[i] < topk) outk[rk4[i]] = mine[i];
            __syncwarp();
            const unsigned long long k = outk[lane];
            if (k != 0ull) { res_v[0] = key_val(k); res_j[0] = key_idx(k); }
            done = true;
        }
    }
    if (!done) {
    // heads of the lists: entry r of CTA c at stv[r * kMaxGrid + c]
    int* stj = reinterpret_cast<int*>(stv) + kMergeDepth * kMaxGrid;
#pragma unroll
    for (int o = 0; o < kMaxOwn; ++o)
#pragma unroll
        for (int r = 0; r < kMergeDepth; ++r) {
            stv[r * kMaxGrid + lane + 32 * o] = ev[r][o];
            stj[r * kMaxGrid + lane + 32 * o] = ej[r][o];
        }
    __syncwarp();
    // k rounds; every lane keeps the current head of each of its lists in registers, a round is two
    // warp reductions, and the winner alone advances (from the staged entries, else from global memory)
    int head[kMaxOwn];
    unsigned long long ck[kMaxOwn];
#pragma unroll
    for (int o = 0; o < kMaxOwn; ++o) {
        head[o] = 0;
        const bool live = (lane + 32 * o < G) && ej[0][o] >= 0;
        ck[o] = live ? key64(ev[0][o], ej[0][o]) : 0ull;
    }
    for (int r = 0; r < topk; ++r) {
        unsigned long long lk = ck[0];
#pragma unroll
        for (int o = 1; o < kMaxOwn; ++o) lk = ck[o] > lk ? ck[o] : lk;
        const unsigned hi = (unsigned)(lk >> 32);
        const unsigned kmax = __reduce_max_sync(0xffffffffu, hi);
        const unsigned lomax = __reduce_max_sync(0xffffffffu, hi == kmax ? (unsigned)lk : 0u);
        if (kmax == 0u) break;                                // every list is exhausted
        const unsigned long long win = ((unsigned long long)kmax << 32) | lomax;
        if (lk == win) {                                      // one lane: advance the list it came from
#pragma unroll
            for (int o = 0; o < kMaxOwn; ++o)
                if (ck[o] == win) {
                    const int c = lane + 32 * o;
                    const int hd = ++head[o];
                    float v = -CUDART_INF_F;
                    int j = -1;
                    if (hd < depth) { v = stv[hd * kMaxGrid + c]; j = stj[hd * kMaxGrid + c]; }
                    else if (hd < topk) {
                        v = ld_cg_f32(recs + rec_at(b, 5 + hd, topk) + c);
                        j = ld_cg_s32(irecs + rec_at(b, 5 + topk + hd, topk) + c);
                    }
                    ck[o] = j >= 0 ? key64(v, j) : 0ull;
                }
        }
        if (lane == (r & 31)) {
            if (r < 32) { res_v[0] = key_val(win); res_j[0] = key_idx(win); }
            else { res_v[1] = key_val(win); res_j[1] = key_idx(win); }
        }
    }
    }
    const int row_w = 1 + topk;
    int* oid = a.out_ids + (size_t)b * row_w;
    float* olp = a.out_logprobs + (size_t)b * row_w;
    bool miss = false;
#pragma unroll
    for (int sl = 0; sl < 2; ++sl) {
        const int r = lane + 32 * sl;
        if (r < topk) {
            const bool ok = row_ok && res_j[sl] >= 0;
            const int id = ok ? (a.map ? __ldg(a.map + res_j[sl]) : res_j[sl]) : -1;
            const float lp = ok ? res_v[sl] - lse : CUDART_NAN_F;
            oid[1 + r] = id;
            olp[1 + r] = lp;
            if (!ok) miss = true;
            if (r == 0 && !a.sampled) { oid[0] = id; olp[0] = lp; }
        }
    }
    bool any_missing = __any_sync(0xffffffffu, miss);
    if (lane == 0) {
        if (a.sampled) {
            const bool ok = row_ok && GJ >= 0;
            oid[0] = ok ? (a.map ? __ldg(a.map + GJ) : GJ) : -1;
            olp[0] = ok ? GZ - lse : CUDART_NAN_F;
            if (!ok) any_missing = true;
        }
        if (a.dbg_lse) a.dbg_lse[b] = lse;
        if (!row_ok) atomicOr(&ctrl->flags, (uint32_t)VT_FLAG_BAD_TEMP);
        else if (any_missing) atomicOr(&ctrl->flags, (uint32_t)VT_FLAG_NAN_ROW);
    }
}

}  // namespace
}  // namespace vt
