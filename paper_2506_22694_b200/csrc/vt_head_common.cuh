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
// staging words (32-bit) per merging warp: staged list heads, selection buffer, output keys (all 64-bit)
constexpr int kMergeStageWords = 2 * (kMergeDepth * kMaxGrid + kSelCap + 64);
constexpr int kStampSlots = 16;                  // phase stamps per CTA (-DVT_STAMPS builds)
#ifdef VT_STAMPS
constexpr size_t kStampBytes = (size_t)kMaxGrid * kStampSlots * 8;
#else
constexpr size_t kStampBytes = 0;
#endif

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
// more than the arithmetic they skip.  No real candidate has key 0, which marks an empty slot.
__device__ __forceinline__ unsigned long long key64(float v, int j) {
    return ((unsigned long long)f2ord(v) << 32) | (unsigned)(~j);
}
__device__ __forceinline__ float key_val(unsigned long long k) { return ord2f((unsigned)(k >> 32)); }
__device__ __forceinline__ int key_idx(unsigned long long k) { return (int)~(unsigned)k; }

// Records.  Per hidden row b a block of rec_fields(topk) * kMaxGrid 32-bit words, laid out in planes
// with the CTA index fastest, so that a merging warp reads every plane with coalesced loads:
//   64-bit planes: 0 = Gumbel-max candidate as key64(score, j); 1 + r = entry r of the CTA's top-k list
//                  as key64(z, j), best first, 0 = no entry;
//   32-bit planes (behind them): 0 = running max m, 1 = sum of exp(z - m), 2 = z of the Gumbel candidate.
__host__ __device__ inline int rec_fields(int topk) { return 5 + 2 * topk; }
__device__ __forceinline__ unsigned long long* rec_keys(float* recs, int b, int topk) {
    return reinterpret_cast<unsigned long long*>(recs + (size_t)b * rec_fields(topk) * kMaxGrid);
}
__device__ __forceinline__ float* rec_f32(float* recs, int b, int topk) {
    return recs + (size_t)b * rec_fields(topk) * kMaxGrid + (size_t)2 * (1 + topk) * kMaxGrid;
}
__device__ __forceinline__ unsigned long long ld_cg_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.global.cg.b64 %0, [%1];" : "=l"(v) : "l"(p));
    return v;
}

struct MergeOut {
    const int32_t* map;
    int32_t* out_ids;
    float* out_logprobs;
    float* dbg_lse;
    int topk;
    int sampled;       // uniforms were given: column 0 is the Gumbel-max draw
};

// A single warp runs dependent code at a few cycles per instruction, so the merge is cut into two
// roles that two warps can run side by side when the CTA has warps to spare:
//   kRoleStats: log-sum-exp over all CTAs, the Gumbel-max winner (column 0 when sampling);
//   kRoleCand : the topk best list entries over all CTAs (columns 1..topk; column 0 when not sampling).
// The candidate log-probabilities need the row's lse: a warp with both roles computes it first; two
// warps sharing a row pass it through `xch` (shared memory) and meet at the named barrier `bar_id`
// (64 threads).  All record loads of a role are issued before their first use.
constexpr int kRoleCand = 1, kRoleStats = 2;

__device__ __noinline__ void merge_records(const MergeOut a, Ctrl* ctrl, float* recs, int b, bool row_ok, int G,
                                           float* stage, int roles, volatile float* xch, int bar_id,
                                           unsigned long long* stamp = nullptr) {
    const int lane = threadIdx.x & 31;
    const int topk = a.topk;
    const unsigned long long* kp = rec_keys(recs, b, topk);
    const float* fp = rec_f32(recs, b, topk);
    const int row_w = 1 + topk;
    int* oid = a.out_ids + (size_t)b * row_w;
    float* olp = a.out_logprobs + (size_t)b * row_w;
    float lse = 0.f;

    // the candidate role's loads go out first in any case
    const int depth = min(topk, kMergeDepth);
    unsigned long long ek[kMergeDepth][kMaxOwn];
    if (roles & kRoleCand) {
#pragma unroll
        for (int r = 0; r < kMergeDepth; ++r)
#pragma unroll
            for (int o = 0; o < kMaxOwn; ++o) {
                const int c = lane + 32 * o;
                ek[r][o] = (c < G && r < depth) ? ld_cg_u64(kp + (size_t)(1 + r) * kMaxGrid + c) : 0ull;
            }
    }

    if (roles & kRoleStats) {
        float hm[kMaxOwn], hs[kMaxOwn], hz[kMaxOwn];
        unsigned long long hk[kMaxOwn];
#pragma unroll
        for (int o = 0; o < kMaxOwn; ++o) {
            const int c = lane + 32 * o;
            const bool on = c < G;
            hm[o] = on ? ld_cg_f32(fp + c) : -CUDART_INF_F;
            hs[o] = on ? ld_cg_f32(fp + kMaxGrid + c) : 0.f;
            hz[o] = (on && a.sampled) ? ld_cg_f32(fp + 2 * kMaxGrid + c) : 0.f;
            hk[o] = (on && a.sampled) ? ld_cg_u64(kp + c) : 0ull;
        }
        // this lane's CTAs in CTA order, then across lanes: the row's maximum by one warp reduction,
        // every lane's sum rescaled to it once, a butterfly of additions (a fixed order: the result does
        // not depend on which CTA finished when)
        float M = -CUDART_INF_F, S = 0.f, gz = 0.f;
        unsigned long long gk = 0ull;
#pragma unroll
        for (int o = 0; o < kMaxOwn; ++o) {
            lse_merge(M, S, hm[o], hs[o]);
            const bool w = hk[o] > gk;
            gk = w ? hk[o] : gk;
            gz = w ? hz[o] : gz;
        }
        const float Mall = ord2f(__reduce_max_sync(0xffffffffu, f2ord(M)));
        float sc = (M == -CUDART_INF_F) ? 0.f : S * __expf(M - Mall);
#pragma unroll
        for (int o = 16; o; o >>= 1) sc += __shfl_xor_sync(0xffffffffu, sc, o);
        lse = Mall + logf(sc);
        if (roles == kRoleStats) {                          // the candidate warp of this row is waiting for it
            if (lane == 0) *xch = lse;
            asm volatile("bar.sync %0, 64;" ::"r"(bar_id) : "memory");
        }
        unsigned long long gwin = 0ull;
        float gzw = 0.f;
        if (a.sampled) {
            const unsigned hi = (unsigned)(gk >> 32);
            const unsigned kmax = __reduce_max_sync(0xffffffffu, hi);
            const unsigned lomax = __reduce_max_sync(0xffffffffu, hi == kmax ? (unsigned)gk : 0u);
            const unsigned who = __ballot_sync(0xffffffffu, hi == kmax && (unsigned)gk == lomax);
            gzw = __shfl_sync(0xffffffffu, gz, __ffs(who) - 1);
            gwin = ((unsigned long long)kmax << 32) | lomax;
        }
        if (lane == 0) {
            bool bad = !(lse == lse);                       // a NaN logit somewhere in the row
            if (a.sampled) {
                const bool ok = row_ok && gwin != 0ull;
                const int gj = key_idx(gwin);
                oid[0] = ok ? (a.map ? __ldg(a.map + gj) : gj) : -1;
                olp[0] = ok ? gzw - lse : CUDART_NAN_F;
                bad = bad || !ok;
            }
            if (a.dbg_lse) a.dbg_lse[b] = lse;
            if (!row_ok) atomicOr(&ctrl->flags, (uint32_t)VT_FLAG_BAD_TEMP);
            else if (bad) atomicOr(&ctrl->flags, (uint32_t)VT_FLAG_NAN_ROW);
        }
    }
    if (!(roles & kRoleCand)) return;
#ifdef VT_STAMPS
    if (stamp && lane == 0 && b == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t) : "l"(ek[0][0] + ek[kMergeDepth - 1][kMaxOwn - 1]));   // after the loads
        stamp[8] = t;
    }
#endif

    unsigned long long res_k[2] = {0ull, 0ull};
    unsigned long long* stk = reinterpret_cast<unsigned long long*>(stage);        // [kMergeDepth][kMaxGrid] list heads
    unsigned long long* sel = stk + kMergeDepth * kMaxGrid;                        // [kSelCap]
    unsigned long long* outk = sel + kSelCap;                                      // [64]
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
            const unsigned h = (unsigned)(ek[0][o] >> 32);
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
        outk[lane] = 0ull;
        outk[lane + 32] = 0ull;
        // compaction: every lane counts its qualifying entries, a warp scan gives it a place to put them
        int mine_n = 0;
        bool deep = false;
#pragma unroll
        for (int r = 0; r < kMergeDepth; ++r)
#pragma unroll
            for (int o = 0; o < kMaxOwn; ++o) {
                const bool in = ek[r][o] != 0ull && (unsigned)(ek[r][o] >> 32) >= tau;
                mine_n += in ? 1 : 0;
                deep = deep || (in && r == depth - 1 && depth < topk);
            }
        int pos = mine_n;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, pos, o);
            pos += (lane >= o) ? y : 0;
        }
        const int n = __shfl_sync(0xffffffffu, pos, 31);
        pos -= mine_n;
        if (n <= kSelCap) {
#pragma unroll
            for (int r = 0; r < kMergeDepth; ++r)
#pragma unroll
                for (int o = 0; o < kMaxOwn; ++o)
                    if (ek[r][o] != 0ull && (unsigned)(ek[r][o] >> 32) >= tau) sel[pos++] = ek[r][o];
        }
        if (n <= kSelCap && !__any_sync(0xffffffffu, deep)) {
            __syncwarp();
            if (n <= 32) {                                                         // the usual case: one entry per lane
                const unsigned long long mine = lane < n ? sel[lane] : 0ull;
                int r1 = 0;
                for (int e = 0; e < n; ++e) r1 += (sel[e] > mine) ? 1 : 0;
                if (lane < n && r1 < topk) outk[r1] = mine;
            } else {
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
            }
            __syncwarp();
            res_k[0] = outk[lane];
            done = true;
        }
    }
    if (!done) {
        // heads of the lists: entry r of CTA c at stk[r * kMaxGrid + c]
#pragma unroll
        for (int o = 0; o < kMaxOwn; ++o)
#pragma unroll
            for (int r = 0; r < kMergeDepth; ++r) stk[r * kMaxGrid + lane + 32 * o] = ek[r][o];
        __syncwarp();
        // k rounds; every lane keeps the current head of each of its lists in registers, a round is two
        // warp reductions, and the winner alone advances (from the staged entries, else from global memory)
        int head[kMaxOwn];
        unsigned long long ck[kMaxOwn];
#pragma unroll
        for (int o = 0; o < kMaxOwn; ++o) {
            head[o] = 0;
            ck[o] = ek[0][o];
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
                        unsigned long long nk = 0ull;
                        if (hd < depth) nk = stk[hd * kMaxGrid + c];
                        else if (hd < topk) nk = ld_cg_u64(kp + (size_t)(1 + hd) * kMaxGrid + c);
                        ck[o] = nk;
                    }
            }
            if (lane == (r & 31)) res_k[r >> 5] = win;
        }
    }
#ifdef VT_STAMPS
    if (stamp && lane == 0 && b == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t) : "l"(res_k[0]));
        stamp[9] = t;
    }
#endif
    // the gathers through the index mapper go out before the wait for the row's lse
    int ids[2];
    float zv[2];
    bool okv[2];
#pragma unroll
    for (int sl = 0; sl < 2; ++sl) {
        const int r = lane + 32 * sl;
        okv[sl] = r < topk && row_ok && res_k[sl] != 0ull;
        const int j = key_idx(res_k[sl]);
        ids[sl] = okv[sl] ? (a.map ? __ldg(a.map + j) : j) : -1;
        zv[sl] = key_val(res_k[sl]);
    }
    if (roles == kRoleCand) {
        asm volatile("bar.sync %0, 64;" ::"r"(bar_id) : "memory");
        lse = *xch;
    }
    bool miss = false;
#pragma unroll
    for (int sl = 0; sl < 2; ++sl) {
        const int r = lane + 32 * sl;
        if (r < topk) {
            const float lp = okv[sl] ? zv[sl] - lse : CUDART_NAN_F;
            oid[1 + r] = ids[sl];
            olp[1 + r] = lp;
            if (!okv[sl]) miss = true;
            if (r == 0 && !a.sampled) { oid[0] = ids[sl]; olp[0] = lp; }
        }
    }
    const bool any_missing = __any_sync(0xffffffffu, miss);
    if (lane == 0 && row_ok && any_missing) atomicOr(&ctrl->flags, (uint32_t)VT_FLAG_NAN_ROW);
#ifdef VT_STAMPS
    if (stamp && lane == 0 && b == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t) :: "memory");   // the stores above needed the gathered ids
        stamp[10] = t;
    }
#endif
}

}  // namespace
}  // namespace vt
