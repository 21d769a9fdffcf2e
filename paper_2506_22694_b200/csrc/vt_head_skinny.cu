// Trimmed LM head for a few hidden rows (B <= 16), fused with its sampling epilogue
// (Algorithm 2, the drafter-forward and index-mapping steps: drafter head over the trimmed vocabulary, then the index mapper).
//
// HBM-bound: the only large operand is W_trim [K,d] bf16, read exactly once.  One persistent CTA
// per SM owns a contiguous slab of vocabulary rows and streams it through a shared-memory ring
// filled by the bulk-copy engine (cp.async.bulk + mbarrier transaction counts): one warp issues,
// besides its share of the math, one multi-kilobyte copy per vocabulary row of a stage (8 rows x
// up to 2048 columns), refilling each stage one step after it was released, so well over 100 KB
// per SM stay in flight whatever the other warps are doing.
//
// Sixteen consumer warps split the hidden dimension.  Each keeps its slice of h in registers as
// ready-made operand fragments and feeds the warp-level tensor instruction mma.m16n8k16 (bf16 in,
// fp32 accumulate) with the hidden rows as the 16-row operand and the stage's 8 vocabulary rows
// as the 8-column operand.  A dot product does not care in which order k is visited, so the 16
// contiguous bytes a lane reads from a W row serve directly as its fragment as long as the h
// fragment is taken from the same k positions.  The tensor instruction only off-loads the FMAs
// (at B = 10 the fp32 pipe could not keep up with HBM); the kernel remains a streaming read.
//
// Per 8-row block the 16 partial tiles meet in shared memory and warp b updates hidden row b, on
// chip: running max / sum-exp of z = logit / T, the row's top-k list, and the Gumbel-max
// candidate from the caller's uniforms.  Logits never go to HBM.  Warps only meet through
// mbarriers (stage full/empty, partial tile full/empty), never through a CTA-wide barrier inside
// the loop.  Each CTA leaves one small record per hidden row; the last CTA to finish (atomic
// ticket, no spinning) merges the records in CTA order, remaps trimmed indices through `map` and
// writes the outputs.  Every wait is bounded: on expiry the CTA raises VT_FLAG_TIMEOUT, drains
// its own copies and leaves.
#include <math_constants.h>

#include "vt_common.cuh"
#include "vt_head_common.cuh"
#include "vt_tree_common.cuh"

namespace vt {

namespace {

constexpr int kNW = 16;                          // consumer warps: split of the hidden dimension
constexpr int kThreads = kNW * 32;
constexpr int kLag = 2;                          // a stage is refilled kLag items after its release
constexpr int kRows = 8;                         // vocabulary rows per stage (mma n)
constexpr int kMaxStages = 8;
constexpr int kMaxB = 16;
constexpr size_t kSmemLimit = 227 * 1024 - 1024; // opt-in limit minus static shared memory
constexpr int kCand = 64;                        // candidate buffer entries per hidden row
constexpr int kSelPerLane = (VT_MAX_TOPK + kCand) / 32;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // default bound of a device-side wait (Ctrl::wait_ns overrides)


// Phase stamps (-DVT_STAMPS builds only): thread 0 of every CTA writes %globaltimer at fixed points into
// a region behind the records; bench.py --case stamps reads them back.  Slots: 0 entry, 1 ring fill
// requested, 2 released by the launch dependency, 3 first stage landed, 4 last stage consumed,
// 5 record written, 6 after the fence, 7 after the ticket, 8-10 merge (loads, selection, outputs), 11 SM id.
#ifdef VT_STAMPS
#define VT_STAMP(slot) do { if (threadIdx.x == 0) stamps[(size_t)blockIdx.x * kStampSlots + (slot)] = global_ns(); } while (0)
#else
#define VT_STAMP(slot) do {} while (0)
#endif

struct Geo {
    int RB;            // row blocks of 8 vocabulary rows
    int S;             // ring stages
    int pitch;         // bytes between rows of a stage (odd multiple of 64: conflict-free 128-bit reads)
    int part_stride;   // floats per warp partial tile
    int ring_bytes;
};

// ---- mbarrier / bulk copy primitives -------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* b, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* b) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* b, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
    return ok != 0;
}
// non-blocking probe of a phase (try_wait may suspend the thread for a system-chosen time before it answers)
__device__ __forceinline__ bool mbar_test(uint64_t* b, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// The bound of a wait is kept with the SM's cycle counter (reading the nanosecond timer costs far more
// than a probe): two cycles per nanosecond, i.e. at least the time asked for at any SM clock up to
// 2 GHz.  It lives in shared memory and is looked at only once a wait has to spin, so it costs the hot
// loop no register.  Bounds under a millisecond spin on non-blocking probes only: try_wait may park the
// warp for a system-chosen time before it answers, which is what a long wait wants and a short bound
// cannot afford.
__device__ __forceinline__ long long bound_cycles(unsigned long long ns) {
    return (long long)(ns < (1ull << 61) ? 2 * ns : (1ull << 62));
}
constexpr long long kShortBoundCycles = 2000000;      // 1 ms
// Bounded wait, called by all 32 lanes of a warp; false when the CTA is aborting or the bound
// expired (which starts an abort).  The outcome is voted on, so the lanes of a warp never part ways
// before a warp-collective instruction (mma, shuffle, ballot).  Inline on purpose: a call here would
// spill the caller's registers at every wait that is not satisfied at once, i.e. at most of them.
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, volatile int* abort_flag,
                                          const volatile long long* bound) {
    bool ok = mbar_test(b, parity);
    if (!ok) {
        const long long t0 = clock64();
        const long long lim = *bound;
        const bool nb = lim < kShortBoundCycles;
        for (;;) {
#pragma unroll 1
            for (int i = 0; i < 64 && !ok; ++i) {
                ok = nb ? mbar_test(b, parity) : mbar_try(b, parity);
                if (nb && clock64() - t0 > lim) break;
            }
            if (ok || *abort_flag) break;
            if (clock64() - t0 > lim) { *abort_flag = 1; break; }
        }
    }
    return __all_sync(0xffffffffu, ok);
}
// bulk copy global -> shared with an L2 eviction-priority hint for the lines it brings in
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint64_t* bar, uint64_t pol) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(pol) : "memory");
}
__device__ __forceinline__ uint4 lds_u4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                         uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct TopkState {
    int cnt;       // entries in the list
    float thr;     // value of entry topk-1 once the list is full, else -inf
};

// Warp-cooperative selection: the best min(topk, cnt + n_c) of a sorted list (tv/tj, cnt entries) and
// a batch of unsorted candidates (cv/cj, n_c entries) become the new sorted list (descending value,
// ties to the lower index).  Every element's final position is its rank -- the number of elements
// that beat it -- so there are no sequential selection rounds: each lane keeps up to kSelPerLane
// elements in registers while all elements stream by as broadcast shared-memory reads.  The cost
// does not depend on topk and is small when few candidates are pending.
template <int NS>
__device__ __forceinline__ void rank_scatter(float* tv, int* tj, int cnt, const float* cv, const int* cj, int n_c,
                                             int topk) {
    const int lane = threadIdx.x & 31;
    const int N = cnt + n_c;
    unsigned long long ek[NS];
    int rk[NS];
#pragma unroll
    for (int i = 0; i < NS; ++i) {
        const int idx = lane + 32 * i;
        ek[i] = 0ull;
        rk[i] = 0;
        if (idx < cnt) ek[i] = key64(tv[idx], tj[idx]);
        else if (idx < N) ek[i] = key64(cv[idx - cnt], cj[idx - cnt]);
    }
#pragma unroll 2
    for (int e = 0; e < cnt; ++e) {
        const unsigned long long k = key64(tv[e], tj[e]);
#pragma unroll
        for (int i = 0; i < NS; ++i) rk[i] += (k > ek[i]) ? 1 : 0;
    }
#pragma unroll 4
    for (int e = 0; e < n_c; ++e) {
        const unsigned long long k = key64(cv[e], cj[e]);
#pragma unroll
        for (int i = 0; i < NS; ++i) rk[i] += (k > ek[i]) ? 1 : 0;
    }
    __syncwarp();                                         // every read of the old list is done
#pragma unroll
    for (int i = 0; i < NS; ++i)
        if (lane + 32 * i < N && rk[i] < topk) { tv[rk[i]] = key_val(ek[i]); tj[rk[i]] = key_idx(ek[i]); }
}

__device__ __noinline__ TopkState topk_flush(float* tv, int* tj, int cnt, const float* cv, const int* cj, int n_c,
                                             int topk) {
    const int N = cnt + n_c;
    __syncwarp();
    if (N <= 32) rank_scatter<1>(tv, tj, cnt, cv, cj, n_c, topk);
    else if (N <= 64) rank_scatter<2>(tv, tj, cnt, cv, cj, n_c, topk);
    else if (N <= 96) rank_scatter<3>(tv, tj, cnt, cv, cj, n_c, topk);
    else rank_scatter<kSelPerLane>(tv, tj, cnt, cv, cj, n_c, topk);
    __syncwarp();
    const int out = min(topk, N);
    return TopkState{out, (out == topk) ? tv[topk - 1] : -CUDART_INF_F};
}

// NCH column chunks per row, KBC 32-column blocks per warp and chunk; TWO: hidden rows 8..15 present.
template <int NCH, int KBC, bool TWO>
__global__ void __launch_bounds__(kThreads, 1)
k_head_stream(const HeadArgs a, Ctrl* ctrl, float* __restrict__ recs, const Geo geo) {
    extern __shared__ __align__(128) uint8_t s_raw[];
    __shared__ uint64_t s_full[kMaxStages], s_empty[kMaxStages], s_pfull[2], s_pempty[2];
    __shared__ int s_last, s_abort, s_any_abort;
    __shared__ long long s_bound;                        // bound of a wait in SM cycles
    __shared__ int s_issued[kMaxStages];                 // per stage: 0 = never requested, else 2 | parity of the latest fill
    __shared__ int s_rowok[kMaxB];                       // per hidden row: its temperature is usable
    __shared__ float s_xch[kMaxB];                       // merge: a row's lse, from its statistics warp to its candidate warp
    constexpr int KC = kNW * KBC * 32;                   // columns per chunk
    const int B = a.B, K = a.K, d = a.d, topk = a.topk;
    const int S = geo.S, pitch = geo.pitch, PT = geo.part_stride;
    const int stage_bytes = kRows * pitch;
    uint8_t* ring = s_raw;
    float* part = reinterpret_cast<float*>(s_raw + geo.ring_bytes);           // [2][kNW][R][PT]
    float* topv = part + 2 * kNW * (TWO ? 2 : 4) * PT;                                        // [B][topk]
    int* topj = reinterpret_cast<int*>(topv + B * topk);                      // [B][topk]
    float* candv = reinterpret_cast<float*>(topj + B * topk);                 // [B][kCand]
    int* candj = reinterpret_cast<int*>(candv + B * kCand);                   // [B][kCand]

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
#ifdef VT_STAMPS
    unsigned long long* stamps = reinterpret_cast<unsigned long long*>(
        reinterpret_cast<uint8_t*>(recs) + align_up_dev((size_t)kMaxGrid * B * rec_fields(topk) * 4, 256));
    if (threadIdx.x == 0) {
        unsigned smid;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        stamps[(size_t)blockIdx.x * kStampSlots + 11] = smid;
    }
#endif
    const int rb0 = (int)((long long)geo.RB * blockIdx.x / gridDim.x);
    const int rb1 = (int)((long long)geo.RB * (blockIdx.x + 1) / gridDim.x);

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(&s_full[s], 1); mbar_init(&s_empty[s], kNW); s_issued[s] = 0; }
        for (int p = 0; p < 2; ++p) { mbar_init(&s_pfull[p], kNW); mbar_init(&s_pempty[p], B); }
        s_abort = 0;
        s_bound = bound_cycles(kWaitLimitNs);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = threadIdx.x; i < B * topk; i += kThreads) { topv[i] = -CUDART_INF_F; topj[i] = -1; }
    __syncthreads();
    VT_STAMP(0);
    volatile int* abort_flag = &s_abort;
    const volatile long long* wait_ns = &s_bound;

    // per-row state of warp b (identical in its four 8-lane groups); declared here so that the
    // record code after the loop sees it
    const int b = warp;
    float invT = 1.f;
    bool row_ok = true;
    float st_m = -CUDART_INF_F, st_s = 0.f;                 // running max / sum exp (per lane)
    float gb_s = -CUDART_INF_F, gb_z = 0.f;                 // Gumbel best (per lane)
    int gb_j = -1;

    // ---- producer duty: one bulk copy per vocabulary row of a stage (lanes 0..7 of the duty warp) ----
    // Every warp tracks the fetch sequence; fetch f is issued by one warp of the duty group (the
    // warps that own no hidden row, so the epilogue warps are spared), in rotation.
    // W_trim is read once per step: its lines are the first to go when L2 needs room, so that the
    // records, the index mapper and h stay resident from step to step
    uint64_t w_policy;                                       // (not volatile: may be re-made where it is used)
    asm("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(w_policy));
    const int n_items = (rb1 - rb0) * NCH;
    const int n_duty = (B < kNW) ? kNW - B : 1;
    int f_item = 0, f_rb = rb0, f_c = 0, f_s = 0, f_duty = kNW - 1;   // next item to fetch, its duty warp
    uint32_t f_ph = 0;
    auto fetch_next = [&]() -> bool {                         // false = abort
        bool ok = true;
        if (warp == f_duty) {
            if (f_item >= S && !mbar_wait(&s_empty[f_s], f_ph ^ 1, abort_flag, wait_ns)) ok = false;
            if (ok) {
                const int nrows = min(kRows, K - f_rb * kRows);
                const int col0 = f_c * KC;
                const uint32_t cbytes = (uint32_t)(min(d, col0 + KC) - col0) * 2u;
                if (lane == 0) {
                    s_issued[f_s] = 2 | (int)f_ph;           // requested at least once; parity of the latest fill
                    mbar_expect_tx(&s_full[f_s], cbytes * (uint32_t)nrows);
                }
                __syncwarp();
                if (lane < nrows)
                    bulk_g2s(smem_u32(ring + (size_t)f_s * stage_bytes + lane * pitch),
                             a.W + (size_t)(f_rb * kRows + lane) * d + col0, cbytes, &s_full[f_s], w_policy);
            }
        }
        ++f_item;
        if (++f_c == NCH) { f_c = 0; ++f_rb; }
        if (++f_s == S) { f_s = 0; f_ph ^= 1; }
        if (--f_duty < kNW - n_duty) f_duty = kNW - 1;
        return ok;
    };
    for (int i = 0; i < S && f_item < n_items; ++i) fetch_next();          // fill the ring (no waits)
    VT_STAMP(1);

    // Programmatic dependent launch (a no-op unless the launch asked for it): the next kernel on the
    // stream may become resident as soon as SMs free up, and this kernel goes no further than
    // fetching weights until everything enqueued before it has completed and is visible.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    VT_STAMP(2);

    // ---- h fragments of this warp's columns, straight from global memory into registers ----------
    uint4 hl[NCH][KBC], hh[NCH][KBC];
#pragma unroll
    for (int c = 0; c < NCH; ++c)
#pragma unroll
        for (int i = 0; i < KBC; ++i) {
            const int col = c * KC + (warp * KBC + i) * 32 + 8 * t;
            hl[c][i] = make_uint4(0, 0, 0, 0);
            hh[c][i] = make_uint4(0, 0, 0, 0);
            if (col < d) {
                if (g < B) hl[c][i] = __ldg(reinterpret_cast<const uint4*>(a.h + (size_t)g * d + col));
                if (TWO && g + 8 < B)
                    hh[c][i] = __ldg(reinterpret_cast<const uint4*>(a.h + (size_t)(g + 8) * d + col));
            }
        }
    {
        const unsigned long long lim = ctrl->wait_ns;        // 0 = the default
        if (lim && threadIdx.x == 0) s_bound = bound_cycles(lim);   // (a race with early waiters only shortens or keeps their bound)
    }
    if (b < B) {
        const float T = a.temp[b];
        row_ok = (T > 0.f) && (T < CUDART_INF_F);
        invT = row_ok ? 1.f / T : CUDART_NAN_F;
        if (lane == 0) s_rowok[b] = row_ok ? 1 : 0;
    }
    float thr = -CUDART_INF_F;                              // k-th best so far (warp uniform)
    int tk_cnt = 0, n_cand = 0;
    const uint32_t lane_off = (uint32_t)(g * pitch + warp * KBC * 64 + t * 16);
    const uint32_t ring_u32 = smem_u32(ring);
    // epilogue lane roles: a group of R row blocks has 8R logits per hidden row; LPR lanes share one
    // logit, each summing the partial tiles of kNW / LPR warps
    constexpr int R = TWO ? 2 : 4;                          // row blocks per exchange
    constexpr int LPR = 4 / R;
    const int e_ri = lane % (8 * R), e_q = lane / (8 * R);
    const int e_r = e_ri >> 3, e_v8 = e_ri & 7;
    float u_next = 0.5f;
    if (a.uniforms && b < B && rb0 + e_r < rb1) {
        const int j = (rb0 + e_r) * kRows + e_v8;
        if (j < K) u_next = __ldg(a.uniforms + (size_t)b * K + j);
    }
    int s = 0, item = 0, n = 0;
    uint32_t ph = 0;
    bool alive = true;
#pragma unroll 1
    for (int rb = rb0; rb < rb1 && alive; rb += R, ++n) {
        const int rc = min(R, rb1 - rb);
        float res[R][TWO ? 4 : 2];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if (r < rc && alive) {
                float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    if (!alive || !mbar_wait(&s_full[s], ph, abort_flag, wait_ns)) { alive = false; continue; }
#ifdef VT_STAMPS
                    if (item == 0) VT_STAMP(3);
#endif
                    const uint32_t base = ring_u32 + (uint32_t)s * (uint32_t)stage_bytes + lane_off;
                    uint4 w[KBC];
#pragma unroll
                    for (int i = 0; i < KBC; ++i) {
                        const int col = c * KC + (warp * KBC + i) * 32 + 8 * t;
                        w[i] = (col < d) ? lds_u4(base + i * 64) : make_uint4(0, 0, 0, 0);
                    }
#pragma unroll
                    for (int i = 0; i < KBC; ++i) {
                        mma_bf16(acc0, hl[c][i].x, hh[c][i].x, hl[c][i].y, hh[c][i].y, w[i].x, w[i].y);
                        mma_bf16(acc1, hl[c][i].z, hh[c][i].z, hl[c][i].w, hh[c][i].w, w[i].z, w[i].w);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&s_empty[s]);
                    if (++s == S) { s = 0; ph ^= 1; }
                    // refill the stage released kLag items ago (by now every warp has normally left it)
                    if (item >= kLag && f_item < n_items && !fetch_next()) alive = false;
                    ++item;
                }
                res[r][0] = acc0[0] + acc1[0];
                res[r][1] = acc0[1] + acc1[1];
                if (TWO) { res[r][2] = acc0[2] + acc1[2]; res[r][3] = acc0[3] + acc1[3]; }
            }
        }
        if (!alive) break;
        // ---- hand the partial tiles over ------------------------------------------------------------
        const int pb = n & 1;
        const uint32_t use = (uint32_t)(n >> 1);
        if (n >= 2 && !mbar_wait(&s_pempty[pb], (use - 1) & 1, abort_flag, wait_ns)) break;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if (r < rc) {
                float* mine = part + ((pb * kNW + warp) * R + r) * PT;
                if (g < B) *reinterpret_cast<float2*>(mine + g * 8 + 2 * t) = make_float2(res[r][0], res[r][1]);
                if (TWO && g + 8 < B)
                    *reinterpret_cast<float2*>(mine + (g + 8) * 8 + 2 * t) = make_float2(res[r][2], res[r][3]);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&s_pfull[pb]);
        if (b >= B) continue;
        // ---- warp b: reduce the tiles, update hidden row b --------------------------------------------
        if (!mbar_wait(&s_pfull[pb], use & 1, abort_flag, wait_ns)) break;
        const bool in_group = e_r < rc;
        float x = 0.f;
        if (in_group) {
            const float* src = part + ((pb * kNW + e_q) * R + e_r) * PT + b * 8 + e_v8;
#pragma unroll
            for (int i = 0; i < kNW / LPR; ++i) x += src[i * LPR * R * PT];
        }
        if (LPR >= 2) x += __shfl_xor_sync(0xffffffffu, x, 8 * R);
        if (LPR >= 4) x += __shfl_xor_sync(0xffffffffu, x, 16 * R);
        __syncwarp();
        if (lane == 0) mbar_arrive(&s_pempty[pb]);
        const int j = (rb + e_r) * kRows + e_v8;
        const bool valid = in_group && j < K;
        if (a.dbg_logits && valid && e_q == 0) a.dbg_logits[(size_t)b * K + j] = x;
        const float z = x * invT;
        {   // online max / sum-exp without a per-lane branch
            const float zz = valid ? z : -CUDART_INF_F;
            const float m_new = fmaxf(st_m, zz);
            const float m_ref = (m_new == -CUDART_INF_F) ? 0.f : m_new;
            st_s = st_s * __expf(st_m - m_ref) + __expf(zz - m_ref);
            st_m = m_new;
        }
        if (a.uniforms) {
            // g = -log(-log u): -log u from a short series in 1-u near 1 (where a fast logarithm's absolute
            // error would dominate the tiny result), fast logarithms elsewhere
            const float uc = fminf(fmaxf(u_next, 0x1p-24f), 1.f - 0x1p-24f);
            const float t1 = 1.f - uc;
            const float lp = t1 * (1.f + t1 * (0.5f + t1 * (0.33333334f + t1 * (0.25f + t1 * 0.2f))));
            const float L = uc > 0.95f ? lp : -__logf(uc);
            const float sc = z - __logf(L);
            if (valid && sc > gb_s) { gb_s = sc; gb_j = j; gb_z = z; }
            const int jn = (rb + R + e_r) * kRows + e_v8;
            if (rb + R + e_r < rb1 && jn < K) u_next = __ldg(a.uniforms + (size_t)b * K + jn);
        }
        const bool is_cand = valid && e_q == 0 && z > thr;
        const unsigned cand = __ballot_sync(0xffffffffu, is_cand);
        if (cand) {
            if (is_cand) {
                const int pos = n_cand + __popc(cand & lanemask_lt());
                candv[b * kCand + pos] = z;
                candj[b * kCand + pos] = j;
            }
            n_cand += __popc(cand);
            if (n_cand + kRows * R > kCand) {
                const TopkState ts = topk_flush(topv + b * topk, topj + b * topk, tk_cnt, candv + b * kCand,
                                                candj + b * kCand, n_cand, topk);
                tk_cnt = ts.cnt;
                thr = ts.thr;
                n_cand = 0;
            }
        }
    }
    VT_STAMP(4);
    // ---- this CTA's record per hidden row ----------------------------------------------------------
    if (b < B && !*abort_flag) {
        if (n_cand > 0) {
            const TopkState ts = topk_flush(topv + b * topk, topj + b * topk, tk_cnt, candv + b * kCand,
                                            candj + b * kCand, n_cand, topk);
            tk_cnt = ts.cnt;
        }
        // Fold the lanes (those sharing a logit hold identical state: only the 8R distinct ones add to the
        // sum): the maximum by one warp reduction, every lane's sum rescaled to it once, a butterfly of
        // additions; the Gumbel candidate by two reductions over its 64-bit key.
        const float Mall = ord2f(__reduce_max_sync(0xffffffffu, f2ord(st_m)));
        float sc = (lane < 8 * (TWO ? 2 : 4) && st_m != -CUDART_INF_F) ? st_s * __expf(st_m - Mall) : 0.f;
#pragma unroll
        for (int o = 16; o; o >>= 1) sc += __shfl_xor_sync(0xffffffffu, sc, o);
        const unsigned long long gk = gb_j >= 0 ? key64(gb_s, gb_j) : 0ull;
        const unsigned ghi = (unsigned)(gk >> 32);
        const unsigned gmax = __reduce_max_sync(0xffffffffu, ghi);
        const unsigned glo = __reduce_max_sync(0xffffffffu, ghi == gmax ? (unsigned)gk : 0u);
        const unsigned who = __ballot_sync(0xffffffffu, ghi == gmax && (unsigned)gk == glo);
        const float gzw = __shfl_sync(0xffffffffu, gb_z, __ffs(who) - 1);
        unsigned long long* kp = rec_keys(recs, b, topk);
        float* fp = rec_f32(recs, b, topk);
        const int c = blockIdx.x;
        if (lane == 0) {
            fp[c] = Mall;
            fp[kMaxGrid + c] = sc;
            fp[2 * kMaxGrid + c] = gzw;
            kp[c] = ((unsigned long long)gmax << 32) | glo;
        }
        for (int r = lane; r < topk; r += 32) {
            const int j = topj[b * topk + r];
            kp[(size_t)(1 + r) * kMaxGrid + c] = j >= 0 ? key64(topv[b * topk + r], j) : 0ull;
        }
        __threadfence();                                    // the record is visible before the ticket is taken
    }
    VT_STAMP(5);
    __syncthreads();                                        // every warp has left the loop: no copy is requested from here on
    VT_STAMP(6);
    if (warp == 0 && *abort_flag) {
        // drain: every stage that was requested must have landed before the CTA may leave
        for (int st = lane; st < S; st += 32) {
            const int last_fill = s_issued[st];
            if (last_fill) {
                const unsigned long long t0 = global_ns();
                while (!mbar_try(&s_full[st], (uint32_t)(last_fill & 1)) && global_ns() - t0 < kWaitLimitNs) {}
            }
        }
        __syncwarp();
    }
    if (threadIdx.x == 0) {
        const bool aborted = s_abort != 0;
        if (aborted) atomicOr(&ctrl->flags, (uint32_t)VT_FLAG_TIMEOUT);
        // Ticket: arrivals in the low half, aborted CTAs in the high half.  Acquire + release in one, so
        // that the last CTA's loads below see every other CTA's record.
        unsigned old;
        asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;"
                     : "=r"(old) : "l"(&ctrl->head_ticket), "r"(aborted ? 0x10001u : 1u) : "memory");
        s_last = ((old & 0xffffu) == gridDim.x - 1);
        s_any_abort = aborted || (old >> 16) != 0;
        if (s_last) ctrl->head_ticket = 0;                  // ready for the next launch
    }
    __syncthreads();
    VT_STAMP(7);
    if (!s_last) return;

    if (s_any_abort) {
        // a bounded wait expired somewhere: the records are incomplete; report every row as missing
        for (int i = threadIdx.x; i < B * (1 + topk); i += kThreads) {
            a.out_ids[i] = -1;
            a.out_logprobs[i] = CUDART_NAN_F;
        }
        return;
    }

    {
        // B <= 8: two warps per hidden row (candidates / statistics) side by side; more rows: one warp each
        const MergeOut mo{a.map, a.out_ids, a.out_logprobs, a.dbg_lse, topk, a.uniforms != nullptr};
        const bool split = B <= kNW / 2;
        const int row = split ? (warp & (kNW / 2 - 1)) : warp;
        const int roles = split ? (warp < kNW / 2 ? kRoleCand : kRoleStats) : (kRoleCand | kRoleStats);
        if (row < B)
            merge_records(mo, ctrl, recs, row, s_rowok[row] != 0, (int)gridDim.x,
                          reinterpret_cast<float*>(ring) + (size_t)row * kMergeStageWords, roles, &s_xch[row], 1 + row
#ifdef VT_STAMPS
                          , stamps + (size_t)blockIdx.x * kStampSlots
#endif
                          );
    }
    if (a.tree.pool_token) {
        // tree drafting: the merged candidates of all rows become pool nodes and the next frontier is
        // chosen here, by the CTA that merged them, instead of in a launch of its own
        __syncthreads();                                   // the rows' outputs are written; the staging area is free
        tree_expand_block(a.tree, a.out_ids, a.out_logprobs, B, topk, 1 + topk, 1,
                          reinterpret_cast<unsigned long long*>(ring), (int)threadIdx.x, kThreads);
    }
}

// ---- host side ---------------------------------------------------------------------------------------
struct Shape {
    int nch, kbc;      // template selection; 0 = unsupported
};

// 32-column blocks per warp needed for d, rounded up to a supported (chunks, blocks per chunk) pair
Shape pick_shape(int d) {
    const int nkb = (d + 31) / 32;
    const int kbw = (nkb + kNW - 1) / kNW;
    static const int table[17][2] = {{0, 0}, {1, 1}, {1, 2}, {1, 3}, {1, 4}, {2, 3}, {2, 3}, {2, 4}, {2, 4},
                                     {3, 3}, {3, 4}, {3, 4}, {3, 4}, {4, 4}, {4, 4}, {4, 4}, {4, 4}};
    if (kbw < 1 || kbw > 16) return Shape{0, 0};
    return Shape{table[kbw][0], table[kbw][1]};
}

bool shape_ok(int B, int d) {
    if (B < 1 || B > kMaxB || d < 8 || (d & 7)) return false;
    const Shape sh = pick_shape(d);
    if (!sh.nch) return false;
    if (B > 8 && sh.nch * sh.kbc > 8) return false;      // h fragments must fit the register file
    return true;
}

Geo make_geo(int B, int K, int d, int topk, size_t* smem_bytes) {
    const Shape sh = pick_shape(d);
    Geo g{};
    g.RB = (K + kRows - 1) / kRows;
    const int kc_bytes = kNW * sh.kbc * 32 * 2;
    g.pitch = kc_bytes + 64;                              // kc_bytes is a multiple of 128
    g.part_stride = ((B * 8 - 8 + 31) / 32) * 32 + 8;     // >= 8 B floats and = 8 (mod 32): conflict-free reduce
    const int R = B > 8 ? 2 : 4;
    const size_t fixed = (size_t)2 * kNW * R * g.part_stride * 4 + (size_t)B * (topk + kCand) * 8;
    const size_t stage = (size_t)kRows * g.pitch;
    int S = (int)((kSmemLimit - fixed) / stage);
    if (S > kMaxStages) S = kMaxStages;
    g.S = S;
    g.ring_bytes = (int)(S * stage);
    *smem_bytes = g.ring_bytes + fixed;
    const size_t merge_bytes = (size_t)B * kMergeStageWords * 4;            // staging area of the merge
    if (*smem_bytes < merge_bytes) *smem_bytes = merge_bytes;
    return g;
}

template <int NCH, int KBC, bool TWO>
cudaError_t launch_variant(const HeadArgs& a, Ctrl* ctrl, float* recs, int grid, const Geo& geo,
                           size_t smem, cudaStream_t s) {
    static int attr_done[64] = {0};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !attr_done[dev]) {
        cudaError_t e = cudaFuncSetAttribute(k_head_stream<NCH, KBC, TWO>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_done[dev] = 1;
    }
    if (a.overlap) {
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)grid);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = s;
        cudaLaunchAttribute attr{};
        attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr.val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        count_launch();
        return cudaLaunchKernelEx(&cfg, k_head_stream<NCH, KBC, TWO>, a, ctrl, recs, geo);
    }
    k_head_stream<NCH, KBC, TWO><<<grid, kThreads, smem, s>>>(a, ctrl, recs, geo);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

bool head_skinny_supported(int32_t B, int32_t d) { return shape_ok(B, d); }

size_t head_skinny_scratch_bytes(int32_t B, int32_t K, int32_t topk) {
    (void)K;
    return align_up((size_t)kMaxGrid * B * rec_fields(topk) * 4, 256) + kStampBytes;
}

#ifdef VT_STAMPS
size_t head_skinny_stamps_offset(int32_t B, int32_t topk) {
    return align_up((size_t)kMaxGrid * B * rec_fields(topk) * 4, 256);
}
#endif

cudaError_t launch_head_skinny(const HeadArgs& a, Ctrl* ctrl, uint8_t* scratch, cudaStream_t s) {
    if (!shape_ok(a.B, a.d)) return cudaErrorInvalidValue;
    size_t smem = 0;
    const Geo geo = make_geo(a.B, a.K, a.d, a.topk, &smem);
    if (geo.S < kLag + 1) return cudaErrorInvalidValue;
    int grid = num_sms();
    if (grid > kMaxGrid) grid = kMaxGrid;
    if (grid > geo.RB) grid = geo.RB;
    float* recs = reinterpret_cast<float*>(scratch);
    const Shape sh = pick_shape(a.d);
    const bool two = a.B > 8;
#define VT_CASE(N, C)                                                                            \
    if (sh.nch == N && sh.kbc == C)                                                              \
        return two ? launch_variant<N, C, true>(a, ctrl, recs, grid, geo, smem, s)               \
                   : launch_variant<N, C, false>(a, ctrl, recs, grid, geo, smem, s);
#define VT_CASE1(N, C)                                                                           \
    if (sh.nch == N && sh.kbc == C) return launch_variant<N, C, false>(a, ctrl, recs, grid, geo, smem, s);
    VT_CASE(1, 1) VT_CASE(1, 2) VT_CASE(1, 3) VT_CASE(1, 4) VT_CASE(2, 3) VT_CASE(2, 4)
    VT_CASE1(3, 3) VT_CASE1(3, 4) VT_CASE1(4, 4)
#undef VT_CASE
#undef VT_CASE1
    return cudaErrorInvalidValue;
}

}  // namespace vt
