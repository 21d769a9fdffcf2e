// Top-K vocabulary selection (Eq. 1, first line: V_trim = V[Top-K(c,k)]) in rank order.
//
// The wanted order -- count descending, equal counts by ascending id -- is exactly what a STABLE
// sort of the ids by descending count produces when it starts from ascending id order.  So the
// whole selection is one least-significant-digit radix sort of V 32-bit counts (8-bit digits,
// passes whose digit is constant are skipped), after which map = first K sorted ids and
// inv_map = rank (or -1) scattered by id.
//
// V is about 1e5: the job is latency-bound, not bandwidth-bound.  It runs as ONE thread-block
// cluster of 8 CTAs (one launch, no grid-wide spin): per pass each CTA counts the digits of its
// contiguous slice, the CTAs exchange their 256 digit totals through distributed shared memory
// between two hardware cluster barriers, and each warp then scatters its sub-slice stably using
// warp match ranks.  Keys and ids ping-pong between two scratch arrays that stay in L2.
#include <cooperative_groups.h>

#include "vt_common.cuh"

namespace cg = cooperative_groups;

namespace vt {

namespace {

constexpr int kCluster = 8;
constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kDigits = 256;
constexpr int kFine = 4096;                      // buckets of the selection pass (3328 in use)
constexpr int kSortCap = 16384;                  // 64-bit keys one CTA ranks in shared memory
constexpr int kCountCap = 2048;                  // largest bucket ranked by counting its greater keys
constexpr uint32_t kWorkCap = 6u << 10;          // key comparisons one CTA spends on that at most, in units of 1024 (~6 K per thread)
constexpr size_t kSelectSmem = sizeof(uint32_t) * 4 * kFine + sizeof(unsigned long long) * kSortCap;
static_assert(sizeof(uint32_t) * 4 * kFine >= sizeof(uint32_t) * kWarps * kDigits, "the full ranking reuses the bucket arrays");

// ---- full ranking: least-significant-digit radix sort over the whole cluster -------------------------
// s_wcnt: [kWarps][kDigits] words of shared memory.
__device__ void lsd_rank_all(cg::cluster_group& cluster, const uint32_t* counts, int32_t V, int32_t K, int32_t* map,
                             int32_t* inv_map, uint32_t* keyA, uint32_t* valA, uint32_t* keyB, uint32_t* valB,
                             uint32_t (*s_wcnt)[kDigits]) {
    const unsigned rank = cluster.block_rank();
    __shared__ uint32_t s_tot[kDigits];            // this CTA's digit totals (read by the peers)
    __shared__ uint32_t s_base[kDigits];           // global start of (digit, this CTA)
    __shared__ uint32_t s_scan[kDigits / 32 + 1];
    __shared__ int s_skip;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nwarps_total = kCluster * kWarps;
    // contiguous sub-slice of each warp, a multiple of 32 long; order = (CTA rank, warp, index)
    const int L = (((V + nwarps_total - 1) / nwarps_total) + 31) & ~31;
    const int gw = rank * kWarps + warp;
    const int lo = min(V, gw * L), hi = min(V, lo + L);

    const uint32_t* src_key = counts;      // pass input: keys; ids are implicit until a scatter ran
    const uint32_t* src_val = nullptr;
    uint32_t* dst_key = keyA;
    uint32_t* dst_val = valA;

    for (int shift = 0; shift < 32; shift += 8) {
        for (int i = threadIdx.x; i < kWarps * kDigits; i += kThreads) (&s_wcnt[0][0])[i] = 0;
        if (threadIdx.x == 0) s_skip = 0;
        __syncthreads();
        // phase 1: digit counts of this warp's sub-slice (descending order: inverted digit)
        for (int i = lo + lane; i < hi; i += 32) {
            const uint32_t dg = 255u - ((src_key[i] >> shift) & 255u);
            atomicAdd(&s_wcnt[warp][dg], 1u);
        }
        __syncthreads();
        if (threadIdx.x < kDigits) {
            uint32_t run = 0;
            for (int w = 0; w < kWarps; ++w) {          // exclusive prefix over the warps
                const uint32_t c = s_wcnt[w][threadIdx.x];
                s_wcnt[w][threadIdx.x] = run;
                run += c;
            }
            s_tot[threadIdx.x] = run;
        }
        cluster.sync();
        // phase 2: global start of every (digit, CTA) from all CTAs' totals
        uint32_t total = 0, before_me = 0;
        if (threadIdx.x < kDigits) {
            for (unsigned c = 0; c < kCluster; ++c) {
                const uint32_t* peer = cluster.map_shared_rank(s_tot, c);
                const uint32_t t = peer[threadIdx.x];
                if (c < rank) before_me += t;
                total += t;
            }
            if (total == (uint32_t)V) s_skip = 1;       // every key has this digit: nothing moves
            // exclusive scan of `total` over the 256 digits (8 warps)
            uint32_t incl = total;
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += y;
            }
            if (lane == 31) s_scan[warp] = incl;
            __syncwarp();
            s_base[threadIdx.x] = incl - total + before_me;   // completed below
        }
        __syncthreads();
        if (threadIdx.x < kDigits) {
            uint32_t off = 0;
            for (int w = 0; w < warp; ++w) off += s_scan[w];
            s_base[threadIdx.x] += off;
        }
        __syncthreads();
        const bool skip = s_skip != 0;
        if (!skip) {
            // phase 3: stable scatter; rank inside the warp's 32 keys by matching digits
            for (int i0 = lo; i0 < hi; i0 += 32) {
                const int i = i0 + lane;
                const bool on = i < hi;
                const unsigned active = __ballot_sync(0xffffffffu, on);
                if (on) {
                    const uint32_t key = src_key[i];
                    const uint32_t val = src_val ? src_val[i] : (uint32_t)i;
                    const uint32_t dg = 255u - ((key >> shift) & 255u);
                    const unsigned peers = __match_any_sync(active, dg);
                    const int leader = __ffs(peers) - 1;
                    uint32_t old = 0;
                    if (lane == leader) {
                        old = s_wcnt[warp][dg];
                        s_wcnt[warp][dg] = old + __popc(peers);
                    }
                    old = __shfl_sync(peers, old, leader);
                    const uint32_t pos = s_base[dg] + old + __popc(peers & lanemask_lt());
                    dst_key[pos] = key;
                    dst_val[pos] = val;
                }
                __syncwarp();
            }
            __threadfence();
        }
        // all CTAs are done reading s_tot and writing dst before anything is reused
        cluster.sync();
        if (!skip) {
            src_key = dst_key;
            src_val = dst_val;
            dst_key = (dst_key == keyA) ? keyB : keyA;
            dst_val = (dst_val == valA) ? valB : valA;
        }
    }
    // emit: sorted position j holds id v
    for (int j = rank * kThreads + threadIdx.x; j < V; j += kCluster * kThreads) {
        const int32_t v = src_val ? (int32_t)src_val[j] : j;
        if (j < K) map[j] = v;
        inv_map[v] = j < K ? j : -1;
    }
}

// Order-preserving bucket of a count: its leading one and the seven bits behind it (counts below 128 map to
// themselves).  3328 buckets whose widths grow with the count, so a heavy-tailed histogram spreads over
// many of them and a bucket near the cut holds a few hundred ids at most.
__device__ __forceinline__ uint32_t fine_bucket(uint32_t c) {
    if (c < 128u) return c;
    const int e = 31 - __clz(c);                                       // 7 .. 31
    return 128u + (uint32_t)(e - 7) * 128u + ((c >> (e - 7)) & 127u);  // 128 .. 3327
}

// Radix select (Eq. 1, Top-K(c,k)): one pass of bucket counts finds the bucket that holds the K-th key;
// only the keys of that bucket and of the buckets above it -- K of them plus part of one bucket -- are
// moved, bucket by bucket, into a scratch array, which is thereby already in bucket order.  Each CTA of
// the cluster then takes a contiguous run of whole buckets into shared memory and gives every key its
// place inside its bucket by counting the bucket's greater keys (64-bit keys (count, ~id): unique, so
// the result is the one right answer; buckets are small, so the counting is cheap).  Everything below
// the cut is never touched again.  When a run does not fit a CTA's shared memory (K close to V) or a
// bucket is too large to rank by counting (counts that all fall into one bucket), the full ranking
// above takes over.
__global__ void __cluster_dims__(kCluster, 1, 1) __launch_bounds__(kThreads, 1)
k_select_sort(const uint32_t* counts, int32_t V, int32_t K, int32_t* map, int32_t* inv_map, uint32_t* keyA, uint32_t* valA, uint32_t* keyB,
              uint32_t* valB) {
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned rank = cluster.block_rank();
    extern __shared__ __align__(16) uint8_t s_dyn[];
    uint32_t* s_hist = reinterpret_cast<uint32_t*>(s_dyn);             // [kFine] this CTA's bucket counts (read by the peers)
    uint32_t* s_gstart = s_hist + kFine;                               // [kFine] start of the bucket in the ranking
    uint32_t* s_gsize = s_gstart + kFine;                              // [kFine] its size over all CTAs
    uint32_t* s_next = s_gsize + kFine;                                // [kFine] scratch position of this CTA's next key
    unsigned long long* s_run = reinterpret_cast<unsigned long long*>(s_next + kFine);     // [kSortCap]
    __shared__ uint32_t s_warp[kWarps + 1];
    __shared__ uint32_t s_load[kCluster];          // keys each CTA would have to rank
    __shared__ uint32_t s_work[kCluster];          // key comparisons that would take: sum of squared bucket sizes, in units of 1024
    __shared__ uint32_t s_T;
    __shared__ int s_cut, s_lo, s_hi, s_big;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // ids of this CTA: a contiguous slice walked with coalesced loads, eight in flight per thread
    const int slice = (V + kCluster - 1) / kCluster;
    const int i0 = min(V, (int)rank * slice), i1 = min(V, i0 + slice);
    constexpr int kInFlight = 8;
    unsigned long long* pairs = reinterpret_cast<unsigned long long*>(keyA);       // [V] 64-bit keys (keyA and valA are adjacent)

    for (int i = threadIdx.x; i < kFine; i += kThreads) s_hist[i] = 0;
    if (threadIdx.x < kCluster) { s_load[threadIdx.x] = 0; s_work[threadIdx.x] = 0u; }
    if (threadIdx.x == 0) { s_cut = 0; s_lo = 0x7fffffff; s_hi = 0; s_big = 0; }
    __syncthreads();
    // phase 1: bucket counts (descending order: inverted bucket index)
    for (int i = i0 + (int)threadIdx.x; i < i1; i += kThreads * kInFlight) {
        uint32_t c[kInFlight];
#pragma unroll
        for (int q = 0; q < kInFlight; ++q) c[q] = i + q * kThreads < i1 ? __ldg(counts + i + q * kThreads) : 0u;
#pragma unroll
        for (int q = 0; q < kInFlight; ++q)
            if (i + q * kThreads < i1) atomicAdd(&s_hist[kFine - 1 - fine_bucket(c[q])], 1u);
    }
    cluster.sync();
    // phase 2: start of every bucket in descending order (each thread owns kFine / kThreads neighbouring
    // buckets), the bucket of the K-th key, who ranks what
    constexpr int BPT = kFine / kThreads;
    static_assert(BPT == 4, "one 128-bit load per peer and thread");
    uint32_t tot[BPT], mine_before[BPT], sum = 0;
#pragma unroll
    for (int q = 0; q < BPT; ++q) { tot[q] = 0; mine_before[q] = 0; }
    uint4 pv[kCluster];
#pragma unroll
    for (unsigned c = 0; c < kCluster; ++c)                         // all eight remote loads in flight
        pv[c] = reinterpret_cast<const uint4*>(cluster.map_shared_rank(s_hist, c))[threadIdx.x];
#pragma unroll
    for (unsigned c = 0; c < kCluster; ++c) {
        const uint32_t t4[BPT] = {pv[c].x, pv[c].y, pv[c].z, pv[c].w};
#pragma unroll
        for (int q = 0; q < BPT; ++q) {
            if (c < rank) mine_before[q] += t4[q];
            tot[q] += t4[q];
        }
    }
#pragma unroll
    for (int q = 0; q < BPT; ++q) sum += tot[q];
    uint32_t incl = sum;
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    uint32_t start = incl - sum;
    for (int w = 0; w < warp; ++w) start += s_warp[w];
#pragma unroll
    for (int q = 0; q < BPT; ++q) {
        const int b = threadIdx.x * BPT + q;
        s_gstart[b] = start;
        s_gsize[b] = tot[q];
        s_next[b] = start + mine_before[q];
        if (start < (uint32_t)K && start + tot[q] >= (uint32_t)K) { s_cut = b; s_T = start + tot[q]; }   // exactly one bucket
        start += tot[q];
    }
    __syncthreads();
    const int cut = s_cut;
    const uint32_t T = s_T;                             // keys to be ranked = end of the cut bucket
#pragma unroll
    for (int q = 0; q < BPT; ++q) {
        const int b = threadIdx.x * BPT + q;
        if (b <= cut && tot[q] > 0) {
            const uint32_t st = s_gstart[b];
            const unsigned owner = min((unsigned)kCluster - 1u, (unsigned)(((unsigned long long)st * kCluster) / T));
            atomicAdd(&s_load[owner], tot[q]);
            if (tot[q] > (uint32_t)kCountCap) s_big = 1;
            else atomicAdd(&s_work[owner], (tot[q] * tot[q] + 1023u) >> 10);
            if (owner == rank) {
                atomicMin(&s_lo, (int)st);
                atomicMax(&s_hi, (int)(st + tot[q]));
            }
        }
    }
    __syncthreads();
    bool fits = s_big == 0;
    for (int c = 0; c < kCluster; ++c) fits = fits && s_load[c] <= (uint32_t)kSortCap && s_work[c] <= kWorkCap;
    if (!fits) {                                        // the same decision in every CTA (same inputs)
        cluster.sync();                                 // peers are done reading this CTA's counts
        lsd_rank_all(cluster, counts, V, K, map, inv_map, keyA, valA, keyB, valB,
                     reinterpret_cast<uint32_t (*)[kDigits]>(s_dyn));
        return;
    }
    // phase 3: move the keys of the buckets down to the cut into bucket order; order inside a bucket is
    // whatever the atomics make of it; ids below the cut are pruned here
    for (int i = i0 + (int)threadIdx.x; i < i1; i += kThreads * kInFlight) {
        uint32_t c[kInFlight];
#pragma unroll
        for (int q = 0; q < kInFlight; ++q) c[q] = i + q * kThreads < i1 ? __ldg(counts + i + q * kThreads) : 0u;
#pragma unroll
        for (int q = 0; q < kInFlight; ++q) {
            const int id = i + q * kThreads;
            if (id >= i1) continue;
            const int b = (int)(kFine - 1 - fine_bucket(c[q]));
            if (b <= cut) pairs[atomicAdd(&s_next[b], 1u)] = ((unsigned long long)c[q] << 32) | (0xffffffffu - (uint32_t)id);
            else inv_map[id] = -1;
        }
    }
    __threadfence();
    cluster.sync();
    // phase 4: this CTA's run of buckets into shared memory; place of a key = start of its bucket + number
    // of greater keys in the bucket (neighbouring lanes mostly share a bucket: the reads are broadcasts)
    const int r0 = s_lo, n = s_hi > s_lo ? s_hi - s_lo : 0;
    for (int j = threadIdx.x; j < n; j += kThreads) s_run[j] = __ldcg(pairs + r0 + j);
    __syncthreads();
    for (int j = threadIdx.x; j < n; j += kThreads) {
        const unsigned long long key = s_run[j];
        const int b = (int)(kFine - 1 - fine_bucket((uint32_t)(key >> 32)));
        const int bs = (int)s_gstart[b] - r0, be = bs + (int)s_gsize[b];
        int r = 0;
        for (int i = bs; i < be; ++i) r += s_run[i] > key ? 1 : 0;
        const int rk = r0 + bs + r;
        const int32_t v = (int32_t)(0xffffffffu - (uint32_t)key);
        if (rk < K) map[rk] = v;
        inv_map[v] = rk < K ? rk : -1;
    }
}

// The full ranking alone, for calls that want (nearly) all of it anyway.
__global__ void __cluster_dims__(kCluster, 1, 1) __launch_bounds__(kThreads, 1)
k_select_full(const uint32_t* counts, int32_t V, int32_t K, int32_t* map, int32_t* inv_map, uint32_t* keyA, uint32_t* valA,
              uint32_t* keyB, uint32_t* valB) {
    cg::cluster_group cluster = cg::this_cluster();
    extern __shared__ __align__(16) uint8_t s_dyn[];
    lsd_rank_all(cluster, counts, V, K, map, inv_map, keyA, valA, keyB, valB, reinterpret_cast<uint32_t (*)[kDigits]>(s_dyn));
}

// Cut of a full ranking at a data-dependent K (the Method section's Top-P and minimum-frequency
// variants of the selection).  `map` holds all V ids in rank order.  mode 0: smallest K whose prefix
// of counts reaches ceil(p * total); mode 1: K = number of ids with count >= min_count.  K is clamped
// to [1, V]; inv_map entries of ranks >= K become -1.  Pure latency (two dependent loads per rank), so
// the ranks are dealt to the 8 CTAs of a cluster, each thread a contiguous run; the CTAs' sums meet
// through distributed shared memory, like the digit totals of the sort.
__global__ void __cluster_dims__(kCluster, 1, 1) __launch_bounds__(kThreads, 1)
k_select_cut(const uint32_t* __restrict__ counts, int32_t V, int mode, double pfrac, uint32_t min_count,
             const int32_t* __restrict__ map, int32_t* __restrict__ inv_map, int32_t* __restrict__ k_out) {
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned rank = cluster.block_rank();
    __shared__ unsigned long long s_part[kThreads];
    __shared__ unsigned long long s_cta_total;          // this CTA's sum (read by the peers)
    __shared__ int s_k;                                 // CTA 0's copy is the cluster's answer
    const int T = kCluster * kThreads;                  // threads of the cluster, in rank order
    const int t = (int)rank * kThreads + (int)threadIdx.x;
    const int per = (V + T - 1) / T;                    // consecutive ranks per thread
    const int j0 = min(V, t * per), j1 = min(V, j0 + per);
    unsigned long long sum = 0;
    int ge = 0;
    for (int j = j0; j < j1; j += 8) {                  // eight ranks (id, then its count) in flight per thread
        int32_t id[8];
        uint32_t c[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) id[q] = j + q < j1 ? map[j + q] : -1;
#pragma unroll
        for (int q = 0; q < 8; ++q) c[q] = id[q] >= 0 ? counts[id[q]] : 0u;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            sum += c[q];
            ge += (id[q] >= 0) & (c[q] >= min_count);
        }
    }
    s_part[threadIdx.x] = mode == 0 ? sum : (unsigned long long)ge;
    if (threadIdx.x == 0) s_k = V;
    __syncthreads();
    if (threadIdx.x < 32) {                             // exclusive scan of this CTA's 1024 partials by one warp
        unsigned long long x[kThreads / 32], run = 0;
#pragma unroll
        for (int q = 0; q < kThreads / 32; ++q) {       // lane l owns partials 32 l .. 32 l + 31
            x[q] = s_part[threadIdx.x * (kThreads / 32) + q];
            run += x[q];
        }
        unsigned long long incl = run;
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long y = __shfl_up_sync(0xffffffffu, incl, o);
            if ((int)threadIdx.x >= o) incl += y;
        }
        unsigned long long pre = incl - run;
#pragma unroll
        for (int q = 0; q < kThreads / 32; ++q) {
            s_part[threadIdx.x * (kThreads / 32) + q] = pre;
            pre += x[q];
        }
        if (threadIdx.x == 31) s_cta_total = incl;
    }
    cluster.sync();                                     // every CTA's total and s_k are in place
    unsigned long long before = 0, total = 0;           // sums of the CTAs before this one / of all
    for (unsigned c = 0; c < kCluster; ++c) {
        const unsigned long long x = *cluster.map_shared_rank(&s_cta_total, c);
        before += c < rank ? x : 0ull;
        total += x;
    }
    int* k_shared = cluster.map_shared_rank(&s_k, 0);
    if (mode == 0) {
        const double target = ceil(pfrac * (double)total);
        unsigned long long cum = before + s_part[threadIdx.x];
        if (t == 0 && target <= 0.0) atomicMin(k_shared, 1);           // an empty histogram: the first rank already reaches it
        // only the thread whose run of ranks crosses the target walks it again
        if ((double)cum < target && (double)(cum + sum) >= target) {
            for (int j = j0; j < j1; ++j) {
                cum += counts[map[j]];
                if ((double)cum >= target) { atomicMin(k_shared, j + 1); break; }
            }
        }
    } else if (t == 0) {
        atomicMin(k_shared, (int)total);
    }
    cluster.sync();                                     // the answer is final; CTA 0 stays until all have read it
    const int K = max(1, min(V, *k_shared));
    if (t == 0) *k_out = K;
    for (int j = K + t; j < V; j += T * 8) {            // eight ids in flight per thread
        int32_t id[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) id[q] = j + q * T < V ? map[j + q * T] : -1;
#pragma unroll
        for (int q = 0; q < 8; ++q)
            if (id[q] >= 0) inv_map[id[q]] = -1;
    }
    cluster.sync();                                     // nobody leaves while a peer may still read its shared memory
}

}  // namespace

cudaError_t launch_select_cut(const uint32_t* counts, int32_t V, int mode, double pfrac, uint32_t min_count,
                              const int32_t* map, int32_t* inv_map, int32_t* k_out, cudaStream_t s) {
    k_select_cut<<<kCluster, kThreads, 0, s>>>(counts, V, mode, pfrac, min_count, map, inv_map, k_out);
    count_launch();
    return cudaGetLastError();
}

size_t select_scratch_bytes(int32_t V) { return 4 * align_up((size_t)V * 4, 256); }

cudaError_t launch_select_topk(const uint32_t* counts, int32_t V, int32_t K, int32_t* map,
                               int32_t* inv_map, uint8_t* scratch, cudaStream_t s) {
    const size_t seg = align_up((size_t)V * 4, 256);
    uint32_t* keyA = reinterpret_cast<uint32_t*>(scratch);
    uint32_t* valA = reinterpret_cast<uint32_t*>(scratch + seg);
    uint32_t* keyB = reinterpret_cast<uint32_t*>(scratch + 2 * seg);
    uint32_t* valB = reinterpret_cast<uint32_t*>(scratch + 3 * seg);
    static int attr_done[64] = {0};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !attr_done[dev]) {
        e = cudaFuncSetAttribute(k_select_sort, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSelectSmem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_done[dev] = 1;
    }
    if ((long long)K * 2 > V)          // more than half the ranking is wanted: rank everything, select nothing
        k_select_full<<<kCluster, kThreads, sizeof(uint32_t) * kWarps * kDigits, s>>>(counts, V, K, map, inv_map, keyA, valA, keyB, valB);
    else
        k_select_sort<<<kCluster, kThreads, kSelectSmem, s>>>(counts, V, K, map, inv_map, keyA, valA, keyB, valB);
    count_launch();
    return cudaGetLastError();
}

}  // namespace vt
