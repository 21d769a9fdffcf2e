// Top-K vocabulary selection (Eq. 1, first line: V_trim = V[Top-K(c,k)]) in rank order, and the Method
// section's two other rules (Top-P, minimum frequency) over the same ranking.
//
// V is about 1e5: the job is latency-bound, not bandwidth-bound.  It runs as ONE thread-block cluster of
// 8 CTAs (one launch, no grid-wide spin) that talk through distributed shared memory between hardware
// cluster barriers.  Two algorithms live here:
//
//  * the selection (k_select_sort, further down): one pass of bucket counts finds where the K-th key lies;
//    only the keys down to there are ranked, and ids that were seen fewer than 1024 times take their
//    rank where they are first placed.  Every call starts here.
//  * the full ranking (lsd_rank_all, first): the wanted order -- count descending, equal counts by
//    ascending id -- is exactly what a STABLE sort of the ids by descending count produces when it
//    starts from ascending id order, so it is one least-significant-digit radix sort of V 32-bit counts
//    (8-bit digits, passes whose digit is constant are skipped): per pass each CTA counts the digits of
//    its contiguous slice, the CTAs exchange their 256 digit totals, and each warp scatters its
//    sub-slice stably using warp match ranks; keys and ids ping-pong between two scratch arrays that stay
//    in L2.  The selection falls through to it when what it would have to rank does not fit its shared
//    memory or would cost more than this.
#include <cooperative_groups.h>

#include "vt_common.cuh"

namespace cg = cooperative_groups;

namespace vt {

namespace {

constexpr int kCluster = 8;
constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kDigits = 256;
constexpr int kFine = 4096;                      // buckets of the selection pass (4032 in use)
constexpr int kSortCap = 12288;                  // keys one CTA ranks in shared memory (a 32-bit short key and a 32-bit rank each)
constexpr int kExact = 1024;                     // counts below this have a bucket to themselves (fine_bucket)
constexpr int kFirstExact = kFine - kExact;      // ... the buckets kFirstExact .. kFine-1 in descending order
constexpr int kExactIds = 65535;                 // ids per CTA up to which such counts are ranked where they are placed (16-bit counters)
constexpr int kCountCap = 2048;                  // largest bucket ranked by counting its greater keys
constexpr uint32_t kWorkCap = 6u << 10;          // key comparisons one CTA spends on that at most, in units of 1024 (~6 K per thread)
constexpr size_t kSelectSmem = sizeof(uint32_t) * 4 * kFine + sizeof(uint32_t) * 2 * kSortCap + sizeof(uint16_t) * (1024 / 32) * kExact;
constexpr int kMassAt = 32 << 10;                // where in the key buffer the buckets' token mass lives while that buffer is idle
static_assert(kMassAt + sizeof(unsigned long long) * kFine <= sizeof(uint32_t) * 2 * kSortCap, "the token mass fits the idle key buffer");
static_assert(sizeof(uint32_t) * (kFine / 8) * (1 + 8) + sizeof(unsigned long long) * (kFine / 8) <= kMassAt, "... behind the exchange's sums");
constexpr int kDeals = 2;                        // ways of dealing the buckets to the CTAs that are tried
constexpr uint32_t kKeyCost0 = 64, kKeyCost1 = 1024;   // comparisons a key is counted as, besides those with its bucket's keys, in each
static_assert(sizeof(uint32_t) * 4 * kFine >= sizeof(uint32_t) * kWarps * kDigits, "the full ranking reuses the bucket arrays");

// What the full ranking needs to find K itself (Top-P / minimum frequency): the cut bucket's ranks
// [first, end) from the bucket pass and what lies before them.
struct CutSpec {
    int mode;                        // 1: Top-P, 2: minimum frequency
    int valid;                       // 0: no cut bucket (no tokens counted, or nothing as frequent as asked): K = 1
    uint32_t first, end;             // ranks of the cut bucket
    unsigned long long mass_before;  // tokens held by the ranks before it
    double target;                   // ceil(p * total)
    uint32_t min_count;
    int32_t* k_out;
};

// ---- full ranking: least-significant-digit radix sort over the whole cluster -------------------------
// s_wcnt: [kWarps][kDigits] words of shared memory.  With `spec`, K is read off the sorted counts before the
// ranking is emitted (every CTA works it out for itself: the same reads, the same answer).
__device__ void lsd_rank_all(cg::cluster_group& cluster, const uint32_t* counts, int32_t V, int32_t K, int32_t* map,
                             int32_t* inv_map, uint32_t* keyA, uint32_t* valA, uint32_t* keyB, uint32_t* valB,
                             uint32_t (*s_wcnt)[kDigits], const CutSpec* spec = nullptr) {
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
    if (spec) {
        __shared__ int s_kfound;
        if (threadIdx.x == 0) s_kfound = 1;
        __syncthreads();
        if (spec->valid && warp == 0) {
            // the sorted counts of the cut bucket's ranks, 32 at a time, until the prefix reaches the target
            // (Top-P) or the counts fall under min_count; equal counts (every bucket under kExact) by division
            const uint32_t a = spec->first, b = spec->end;
            const uint32_t c0 = src_key[a];
            int found = (int)b;                                        // (the bucket pass says the cut lies in [a, b])
            if (spec->mode == 1 && c0 < (uint32_t)kExact) {
                const unsigned long long rem = (unsigned long long)spec->target - spec->mass_before;
                found = (int)(a + (uint32_t)((rem + c0 - 1) / c0));
            } else {
                unsigned long long cum = spec->mass_before;
                bool done = false;
                for (uint32_t j0 = a; j0 < b && !done; j0 += 32) {
                    const uint32_t j = j0 + lane;
                    const uint32_t c = j < b ? src_key[j] : 0u;
                    if (spec->mode == 1) {
                        unsigned long long incl = c;
                        for (int o = 1; o < 32; o <<= 1) {
                            const unsigned long long y = __shfl_up_sync(0xffffffffu, incl, o);
                            if (lane >= o) incl += y;
                        }
                        const unsigned hit = __ballot_sync(0xffffffffu, j < b && (double)(cum + incl) >= spec->target);
                        if (hit) { found = (int)(j0 + __ffs(hit)); done = true; }
                        cum += __shfl_sync(0xffffffffu, incl, 31);
                    } else {
                        const unsigned low = __ballot_sync(0xffffffffu, j >= b || c < spec->min_count);
                        if (low) { found = (int)(j0 + __ffs(low) - 1); done = true; }
                    }
                }
            }
            if (lane == 0) s_kfound = max(1, min(V, found));
        }
        __syncthreads();
        K = s_kfound;
        if (rank == 0 && threadIdx.x == 0) *spec->k_out = K;
    }
    // emit: sorted position j holds id v
    for (int j = rank * kThreads + threadIdx.x; j < V; j += kCluster * kThreads) {
        const int32_t v = src_val ? (int32_t)src_val[j] : j;
        if (j < K) map[j] = v;
        inv_map[v] = j < K ? j : -1;
    }
}

// The keys of one bucket of counts >= 1024 agree in the count's leading one and the five to nine bits behind it; what
// orders them is the rest of the count and then ~id.  Where that fits 32 bits (lb low bits of the count + the
// bits of an id) it is the short key compared in shared memory; a bucket where it does not fit (counts from 2^21
// with a 17-bit id) is called wide and compares its 64-bit keys where they lie in global memory -- the deal
// hands such a bucket to the ranking only while it is tiny.
__device__ __forceinline__ int id_bits(int32_t V) { return 32 - __clz(max(V - 1, 1)); }          // 1 .. 31
// Bits of a count that its bucket leaves open, from the count and from the bucket (ascending index).
__device__ __forceinline__ int low_bits(uint32_t cnt) {
    if (cnt < (uint32_t)kExact) return 0;
    const int e = 31 - __clz(cnt);
    return e < 14 ? e - 9 : e < 18 ? e - 7 : e - 5;                                        // 1 .. 26
}
__device__ __forceinline__ int low_bits_of_bucket(int asc) {
    if (asc < kExact) return 0;
    if (asc < 3072) return 10 + (asc - 1024) / 512 - 9;
    if (asc < 3584) return 14 + (asc - 3072) / 128 - 7;
    return 18 + (asc - 3584) / 32 - 5;
}
__device__ __forceinline__ uint32_t short_key(unsigned long long key, int idbits) {
    const uint32_t cnt = (uint32_t)(key >> 32);
    const int lb = low_bits(cnt);
    if (lb + idbits > 32) return 0u;
    return ((cnt & ((1u << lb) - 1u)) << idbits) | ((uint32_t)key & ((1u << idbits) - 1u));       // (~id in idbits bits)
}
constexpr uint32_t kWideCap = 32;                // ids a wide bucket may hold and still be ranked by counting

// Number of keys of the bucket [bs, be) of the CTA's run that are greater than key (and, MASS, the sum of their counts).
template <bool MASS>
__device__ __forceinline__ int rank_in_bucket(const uint32_t* s_c, const unsigned long long* run, unsigned long long key, int bs, int be,
                                              int idbits, unsigned long long* mass) {
    const uint32_t cnt = (uint32_t)(key >> 32);
    const int lb = low_bits(cnt);
    int r = 0;
    if (lb + idbits > 32) {                          // wide bucket
        unsigned long long m = 0;
        for (int i = bs; i < be; ++i) {
            const unsigned long long o = __ldcg(run + i);
            const bool gt = o > key;
            r += gt ? 1 : 0;
            if (MASS) m += gt ? (o >> 32) : 0ull;
        }
        if (MASS) *mass = m;
        return r;
    }
    const uint32_t ck = short_key(key, idbits);
    if (MASS) {
        unsigned long long m = 0;                    // of the counts' low bits
        for (int i = bs; i < be; ++i) {
            const uint32_t o = s_c[i];
            const bool gt = o > ck;
            r += gt ? 1 : 0;
            m += gt ? (unsigned long long)(o >> idbits) : 0ull;
        }
        *mass = (unsigned long long)r * (cnt & ~((1u << lb) - 1u)) + m;
        return r;
    }
    int i = bs;
    for (; i < be && (i & 3); ++i) r += s_c[i] > ck ? 1 : 0;
    for (; i + 4 <= be; i += 4) {
        const uint4 o = *reinterpret_cast<const uint4*>(s_c + i);
        r += (o.x > ck ? 1 : 0) + (o.y > ck ? 1 : 0) + (o.z > ck ? 1 : 0) + (o.w > ck ? 1 : 0);
    }
    for (; i < be; ++i) r += s_c[i] > ck ? 1 : 0;
    return r;
}

// Order-preserving bucket of a count: counts below 1024 map to themselves; above that the leading one and the
// bits behind it pick the bucket -- nine bits for counts below 2^14 (where the cut of a large corpus falls and a
// bucket would otherwise hold hundreds of ids), seven below 2^18, five above (a few hundred ids in all at such
// counts).  4032 buckets whose widths grow with the count, so a heavy-tailed histogram spreads over many of them.
__device__ __forceinline__ uint32_t fine_bucket(uint32_t c) {
    // (no branches: the bits of c converted to fp32 toward zero are its exponent followed by the bits behind the
    // leading one, so a shift leaves exponent and m bits, and the octave's first bucket is a constant away)
    const uint32_t bits = __float_as_uint(__uint2float_rz(c));
    const bool lo = c < (1u << 14), mid = c < (1u << 18);
    const uint32_t sh = lo ? 14u : mid ? 16u : 18u;                    // 23 - m
    const uint32_t off = lo ? 69120u : mid ? 14976u : 1056u;           // ((127 + first e) << m) - first bucket of the range
    return c < (uint32_t)kExact ? c : (bits >> sh) - off;              // 1024..3071 | 3072..3583 | 3584..4031
}

// Radix select (Eq. 1, Top-K(c,k)): one pass of bucket counts finds the bucket that holds the K-th key;
// only the keys of that bucket and of the buckets above it -- K of them plus part of one bucket -- are
// moved, bucket by bucket, into a scratch array, which is thereby already in bucket order.  Each CTA of
// the cluster then takes a contiguous run of whole buckets and gives every key its place inside its
// bucket by counting the bucket's greater keys (keys (count, ~id) are unique, so the result is the one
// right answer; buckets are small, so the counting is cheap; what is compared is the 32-bit short key
// above, held in shared memory).  Everything below the cut is never touched again.  When no deal of the
// buckets fits the CTAs' shared memory (K close to V on counts that are mostly above 255) or a bucket is
// too large to rank by counting (counts that all fall into one bucket), the full ranking above takes over.
//
// Counts under kExact are the exception to all of that.  Their buckets hold one value each, so inside them the
// order is the order of the ids -- and they are the large ones (thousands of ids that were seen once or twice in a
// small calibration corpus).  Such an id gets its final rank when it is first placed: start of the bucket + ids of the
// bucket in the CTAs before this one + ids of the bucket in the warps before this one (per-warp counts from the
// counting pass, warps walk contiguous pieces of the CTA's slice) + its place among the warp's 32 ids (match.any).
// It is emitted on the spot and never enters the key buffer, whatever the size of its bucket.
//
// MODE 1 / 2 (the Method section's Top-P and minimum-frequency rules): K is not given but found on the way.
// The bucket pass also sums the token mass of every bucket (Top-P), the cut bucket is the one in which the
// prefix mass reaches ceil(p * total) / the one min_count falls into, everything down to the end of that
// bucket is ranked as above, and the CTA that ranks the cut bucket reads K off the ranks (the key whose
// prefix mass crosses the target / the number of keys with count >= min_count) before anything is
// emitted.  map[0, K) and inv_map are written; k_out receives K.  When the run does not fit (see above) or
// the histogram is degenerate (no tokens, nothing down to the cut), the full ranking takes over here too and
// reads K off the sorted counts of the cut bucket's ranks.
template <int MODE>
__global__ void __cluster_dims__(kCluster, 1, 1) __launch_bounds__(kThreads, 1)
k_select_sort(const uint32_t* counts, int32_t V, int32_t K, int32_t* map, int32_t* inv_map, uint32_t* keyA, uint32_t* valA, uint32_t* keyB,
              uint32_t* valB, double pfrac, uint32_t min_count, int32_t* k_out) {
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned rank = cluster.block_rank();
    extern __shared__ __align__(16) uint8_t s_dyn[];
    uint32_t* s_hist = reinterpret_cast<uint32_t*>(s_dyn);             // [kFine] this CTA's bucket counts (read by the peers)
    uint32_t* s_gstart = s_hist + kFine;                               // [kFine] start of the bucket in the ranking
    uint32_t* s_gsize = s_gstart + kFine;                              // [kFine] its size over all CTAs
    uint32_t* s_next = s_gsize + kFine;                                // [kFine] scratch position of this CTA's next key
    unsigned long long* s_run = reinterpret_cast<unsigned long long*>(s_next + kFine);     // [kSortCap] phase 2: the exchange; phase 4: short keys, ranks
    uint16_t (*s_ws)[kExact] = reinterpret_cast<uint16_t (*)[kExact]>(s_run + kSortCap);   // [kWarps][kExact] ids of a warp's piece per exact count
    uint32_t* s_ws2 = reinterpret_cast<uint32_t*>(&s_ws[0][0]);        // ... two counters to a word for the atomics
    // MODE 1: token mass of the buckets (read by the peers), in the key buffer while that is idle: the sums of the counts'
    // low and high 16 bits, which cannot pass 32 bits for a slice of kExactIds ids; beyond that one 64-bit sum (a slow add)
    uint32_t* s_mlo = reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(s_run) + kMassAt);   // [kFine]
    uint32_t* s_mhi = s_mlo + kFine;                                                              // [kFine]
    unsigned long long* s_mass = reinterpret_cast<unsigned long long*>(s_mlo);                    // [kFine] instead of the two
    __shared__ uint32_t s_warp[kWarps + 1];
    __shared__ unsigned long long s_wmass[kWarps + 1];
    __shared__ unsigned long long s_mass_before;    // token mass of the buckets above the cut
    __shared__ int s_cut_owner[kDeals], s_K, s_first;
    __shared__ uint32_t s_load[kDeals][kCluster];  // keys each CTA would have to rank, per way of dealing the buckets
    __shared__ uint32_t s_work[kDeals][kCluster];  // key comparisons that would take: sum of squared bucket sizes, in units of 1024
    __shared__ uint32_t s_T;
    __shared__ int s_cut, s_lo[kDeals], s_hi[kDeals], s_big;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // ids of this CTA: a contiguous slice; every warp walks a contiguous piece of it in id order (128 bytes per
    // load instruction), sixteen loads in flight per lane (all of a lane's ids at V = 128256)
    const int slice = (V + kCluster - 1) / kCluster;
    const int i0 = min(V, (int)rank * slice), i1 = min(V, i0 + slice);
    const bool exact_on = slice <= kExactIds;           // (beyond that every count is ranked through the key buffer)
    const int first_exact = exact_on ? kFirstExact : kFine;
    constexpr int kInFlight = 16;
    const int piece = (((slice + kWarps - 1) / kWarps) + 31) & ~31;
    const int w0 = min(i1, i0 + warp * piece), w1 = min(i1, w0 + piece);
    unsigned long long* pairs = reinterpret_cast<unsigned long long*>(keyA);       // [V] 64-bit keys (keyA and valA are adjacent)

    for (int i = threadIdx.x; i < kFine; i += kThreads) {
        s_hist[i] = 0;
        if (MODE == 1) s_mass[i] = 0ull;
    }
    for (int i = threadIdx.x; i < kWarps * kExact / 8; i += kThreads) reinterpret_cast<uint4*>(s_ws2)[i] = make_uint4(0, 0, 0, 0);
    if (threadIdx.x < kDeals * kCluster) { (&s_load[0][0])[threadIdx.x] = 0; (&s_work[0][0])[threadIdx.x] = 0u; }
    if (threadIdx.x < kDeals) { s_lo[threadIdx.x] = 0x7fffffff; s_hi[threadIdx.x] = 0; s_cut_owner[threadIdx.x] = -1; }
    if (threadIdx.x == 0) { s_cut = -1; s_big = 0; s_K = 0; s_first = 0; s_T = 0; s_mass_before = 0; }
    __syncthreads();
    // phase 1: bucket counts (descending order: inverted bucket index), and per warp the ids of every exact count
    for (int i = w0 + lane; i < w1; i += 32 * kInFlight) {
        uint32_t c[kInFlight];
#pragma unroll
        for (int q = 0; q < kInFlight; ++q) c[q] = i + q * 32 < w1 ? __ldg(counts + i + q * 32) : 0u;
#pragma unroll
        for (int q = 0; q < kInFlight; ++q)
            if (i + q * 32 < w1) {
                const uint32_t b = kFine - 1 - fine_bucket(c[q]);
                if (exact_on && c[q] < (uint32_t)kExact)            // (a warp's piece is 2048 ids at most: no carry between the halves;
                    atomicAdd(&s_ws2[(warp * kExact + (int)c[q]) >> 1], 1u << ((c[q] & 1u) * 16u));   // the bucket's count is their sum, below)
                else
                    atomicAdd(&s_hist[b], 1u);
                if (MODE == 1 && c[q] >= (uint32_t)kExact) {        // (a bucket under kExact holds one value: its mass is a product)
                    if (exact_on) {
                        atomicAdd(&s_mlo[b], c[q] & 0xffffu);
                        atomicAdd(&s_mhi[b], c[q] >> 16);
                    } else {
                        atomicAdd(&s_mass[b], (unsigned long long)c[q]);
                    }
                }
            }
    }
    __syncthreads();
    if (exact_on && threadIdx.x < kExact / 2) {         // exclusive prefix over the warps, per exact count, two counts to a word
        uint32_t t[kWarps], run = 0;                    // (at most kExactIds ids in the CTA's slice: no carry between the halves)
#pragma unroll
        for (int w = 0; w < kWarps; ++w) t[w] = s_ws2[w * (kExact / 2) + threadIdx.x];
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            s_ws2[w * (kExact / 2) + threadIdx.x] = run;
            run += t[w];
        }
        s_hist[kFine - 1 - 2 * (int)threadIdx.x] = run & 0xffffu;       // the CTA's ids with count 2t and 2t + 1
        s_hist[kFine - 2 - 2 * (int)threadIdx.x] = run >> 16;
    }
    cluster.sync();
    // phase 2: start of every bucket in descending order (each thread owns kFine / kThreads neighbouring
    // buckets), the bucket of the K-th key, who ranks what
    constexpr int BPT = kFine / kThreads;
    static_assert(BPT == 4, "one 128-bit load per peer and thread");
    // The eight CTAs' counts meet in two steps, so that 48 KB instead of 128 KB cross between the SMs per CTA: CTA r
    // adds up the buckets [r * kSlice, (r + 1) * kSlice) of all eight (and, per peer, what the peers before it hold),
    // leaves the sums in its own shared memory (the key buffer is idle until the ranking), and after one more cluster
    // barrier every CTA reads the totals and its own row of the prefix table from the bucket's summing CTA.
    constexpr int kSlice = kFine / kCluster;                         // buckets summed by one CTA
    uint32_t* s_tot = reinterpret_cast<uint32_t*>(s_run);            // [kSlice] totals of this CTA's slice
    uint32_t* s_pre = s_tot + kSlice;                                // [kCluster][kSlice] counts held by the peers before peer c
    unsigned long long* s_mtot = reinterpret_cast<unsigned long long*>(s_pre + kCluster * kSlice);   // [kSlice] token mass (MODE 1)
    if (threadIdx.x < kSlice / BPT) {
        const int i4 = (int)rank * (kSlice / BPT) + (int)threadIdx.x;   // which 128-bit group of the bucket arrays
        uint4 pv[kCluster];
#pragma unroll
        for (unsigned c = 0; c < kCluster; ++c)                     // all eight remote loads in flight
            pv[c] = reinterpret_cast<const uint4*>(cluster.map_shared_rank(s_hist, c))[i4];
        uint4 run = make_uint4(0, 0, 0, 0);
#pragma unroll
        for (unsigned c = 0; c < kCluster; ++c) {
            reinterpret_cast<uint4*>(s_pre + c * kSlice)[threadIdx.x] = run;
            run.x += pv[c].x; run.y += pv[c].y; run.z += pv[c].z; run.w += pv[c].w;
        }
        reinterpret_cast<uint4*>(s_tot)[threadIdx.x] = run;
        if (MODE == 1) {
            unsigned long long m4[BPT] = {0, 0, 0, 0};
#pragma unroll
            for (unsigned c = 0; c < kCluster; ++c) {
                if (exact_on) {
                    const uint4 lo4 = reinterpret_cast<const uint4*>(cluster.map_shared_rank(s_mlo, c))[i4];
                    const uint4 hi4 = reinterpret_cast<const uint4*>(cluster.map_shared_rank(s_mhi, c))[i4];
                    m4[0] += (unsigned long long)lo4.x + ((unsigned long long)hi4.x << 16);
                    m4[1] += (unsigned long long)lo4.y + ((unsigned long long)hi4.y << 16);
                    m4[2] += (unsigned long long)lo4.z + ((unsigned long long)hi4.z << 16);
                    m4[3] += (unsigned long long)lo4.w + ((unsigned long long)hi4.w << 16);
                } else {
                    const ulonglong2* mp = reinterpret_cast<const ulonglong2*>(cluster.map_shared_rank(s_mass, c)) + i4 * 2;
                    const ulonglong2 ma = mp[0], mb = mp[1];
                    m4[0] += ma.x; m4[1] += ma.y; m4[2] += mb.x; m4[3] += mb.y;
                }
            }
#pragma unroll
            for (int q = 0; q < BPT; ++q) s_mtot[threadIdx.x * BPT + q] = m4[q];
        }
    }
    cluster.sync();
    uint32_t tot[BPT], mine_before[BPT], sum = 0;
    unsigned long long mass[BPT], msum = 0;
    {
        const unsigned summer = threadIdx.x / (kSlice / BPT);        // the CTA that summed this thread's buckets
        const int i4 = (int)threadIdx.x % (kSlice / BPT);
        const uint4 t4 = reinterpret_cast<const uint4*>(cluster.map_shared_rank(s_tot, summer))[i4];
        const uint4 p4 = reinterpret_cast<const uint4*>(cluster.map_shared_rank(s_pre, summer) + rank * kSlice)[i4];
        tot[0] = t4.x; tot[1] = t4.y; tot[2] = t4.z; tot[3] = t4.w;
        mine_before[0] = p4.x; mine_before[1] = p4.y; mine_before[2] = p4.z; mine_before[3] = p4.w;
#pragma unroll
        for (int q = 0; q < BPT; ++q) { sum += tot[q]; mass[q] = 0; }
        if (MODE == 1) {
            const ulonglong2* mp2 = reinterpret_cast<const ulonglong2*>(cluster.map_shared_rank(s_mtot, summer) + i4 * BPT);
            const ulonglong2 ma = mp2[0], mb = mp2[1];
            const unsigned long long mp[BPT] = {ma.x, ma.y, mb.x, mb.y};
#pragma unroll
            for (int q = 0; q < BPT; ++q) {
                const uint32_t value = (uint32_t)(kFine - 1 - (threadIdx.x * BPT + q));      // the bucket's count when under kExact
                mass[q] = value < (uint32_t)kExact ? (unsigned long long)value * tot[q] : mp[q];
                msum += mass[q];
            }
        }
    }
    unsigned long long mincl = msum;
    if (MODE == 1) {
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long y = __shfl_up_sync(0xffffffffu, mincl, o);
            if (lane >= o) mincl += y;
        }
        if (lane == 31) s_wmass[warp] = mincl;
    }
    uint32_t incl = sum;
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    uint32_t start = incl - sum;
    for (int w = 0; w < warp; ++w) start += s_warp[w];
    unsigned long long mstart = mincl - msum, mtotal = 0;
    // Top-P: target = ceil(p * total) is the one fp64 product; what is compared with it are integers, and while the
    // total is under 2^53 (every prefix then converts exactly) they are compared as integers -- fp64 conversions of
    // every bucket's prefix in every thread were 5 us of this kernel
    double target = 0.0;
    unsigned long long itarget = 0;
    bool as_int = true;
    if (MODE == 1) {
        for (int w = 0; w < warp; ++w) mstart += s_wmass[w];
        for (int w = 0; w < kWarps; ++w) mtotal += s_wmass[w];
        if (lane == 0) target = ceil(pfrac * (double)mtotal);
        target = __shfl_sync(0xffffffffu, target, 0);
        as_int = mtotal < (1ull << 53);
        itarget = as_int ? (unsigned long long)target : 0ull;
    }
    auto below = [&](unsigned long long x) { return as_int ? x < itarget : (double)x < target; };
    auto reaches = [&](unsigned long long x) { return as_int ? x >= itarget : (double)x >= target; };
    const int min_bucket = MODE == 2 ? (int)(kFine - 1 - fine_bucket(min_count)) : 0;
#pragma unroll
    for (int q = 0; q < BPT; ++q) {
        const int b = threadIdx.x * BPT + q;
        s_gstart[b] = start;
        s_gsize[b] = tot[q];
        s_next[b] = start + mine_before[q];
        bool is_cut;
        if (MODE == 0) is_cut = start < (uint32_t)K && start + tot[q] >= (uint32_t)K;                   // exactly one bucket
        else if (MODE == 1) is_cut = below(mstart) && reaches(mstart + mass[q]);                       // exactly one, if any token was counted
        else is_cut = b == min_bucket;
        if (is_cut) {
            s_cut = b; s_T = start + tot[q]; s_mass_before = mstart; s_K = (int)start; s_first = (int)start;
            if (MODE != 0 && b >= first_exact) {        // an exact bucket: K follows by arithmetic, here and now
                const uint32_t value = (uint32_t)(kFine - 1 - b);
                uint32_t kk;
                if (MODE == 1) kk = start + (uint32_t)(((unsigned long long)target - mstart + value - 1) / value);
                else kk = start + tot[q];               // (the bucket min_count falls into holds exactly min_count)
                s_K = (int)max(1u, min((uint32_t)V, kk));
                if (rank == 0) *k_out = s_K;
            }
        }
        start += tot[q];
        mstart += mass[q];
    }
    __syncthreads();
    const int cut = s_cut;
    const uint32_t T = s_T;                             // keys to be ranked = end of the cut bucket
    CutSpec spec{MODE, cut >= 0 && T > 0, (uint32_t)s_first, T, s_mass_before, target, min_count, k_out};
    if (MODE != 0 && !spec.valid) {                     // no tokens at all / nothing as frequent as asked: K = 1 of the full ranking
        cluster.sync();                                 // peers are done reading this CTA's counts
        lsd_rank_all(cluster, counts, V, V, map, inv_map, keyA, valA, keyB, valB,
                     reinterpret_cast<uint32_t (*)[kDigits]>(s_dyn), &spec);
        return;
    }
    // Who ranks what: contiguous runs of whole buckets with equal COST, not equal key counts -- a key's place costs
    // one comparison per key of its bucket, so the wide buckets of small counts near the cut dominate (dealt by
    // keys, one CTA ranked for 22 us while another was done in 5).  cost(bucket) = size * (size + key cost); the
    // linear term stands for the per-key work and keeps a run of tiny buckets from outgrowing shared memory.
    // Two deals are tried and the first that fits is taken: the second, with a higher key cost and so closer to
    // equal key counts, is for rankings of 50 K keys and more, where the first one's leading CTA would get more
    // tiny buckets than its shared memory holds.
    int deal = -1;
    for (int d = 0; d < kDeals && deal < 0; ++d) {      // (the same trips in every thread of every CTA: same inputs)
        const uint32_t kc = d == 0 ? kKeyCost0 : kKeyCost1;
        uint32_t cost[BPT], csum = 0;
#pragma unroll
        for (int q = 0; q < BPT; ++q) {
            const int b = threadIdx.x * BPT + q;
            const uint32_t sz = (b <= cut && b < first_exact) ? tot[q] : 0u;    // (ids of exact buckets are placed directly)
            cost[q] = sz * (min(sz, (uint32_t)kCountCap) + kc);                 // (<= 128 K keys in all: the sum fits 32 bits)
            csum += cost[q];
        }
        uint32_t cincl = csum;
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xffffffffu, cincl, o);
            if (lane >= o) cincl += y;
        }
        if (lane == 31) s_warp[warp] = cincl;            // (a barrier lies between this and the last reads of the array)
        __syncthreads();
        uint32_t cstart = cincl - csum, ctotal = 0;
        for (int w = 0; w < kWarps; ++w) {
            if (w < warp) cstart += s_warp[w];
            ctotal += s_warp[w];
        }
#pragma unroll
        for (int q = 0; q < BPT; ++q) {
            const int b = threadIdx.x * BPT + q;
            if (b <= cut && b < first_exact && tot[q] > 0) {
                const uint32_t st = s_gstart[b];
                const int lb = low_bits_of_bucket(kFine - 1 - b);
                if (tot[q] > (uint32_t)kCountCap || (lb + id_bits(V) > 32 && tot[q] > kWideCap)) s_big = 1;
                const unsigned owner = min((unsigned)kCluster - 1u, (unsigned)(((unsigned long long)cstart * kCluster) / max(ctotal, 1u)));
                atomicAdd(&s_load[d][owner], tot[q]);
                if (tot[q] <= (uint32_t)kCountCap) atomicAdd(&s_work[d][owner], (tot[q] * tot[q] + 1023u) >> 10);
                if (owner == rank) {
                    atomicMin(&s_lo[d], (int)st);
                    atomicMax(&s_hi[d], (int)(st + tot[q]));
                }
                if (b == cut) s_cut_owner[d] = (int)owner;
            }
            cstart += cost[q];
        }
        __syncthreads();
        bool ok = s_big == 0;
        for (int c = 0; c < kCluster; ++c) ok = ok && s_load[d][c] <= (uint32_t)kSortCap && s_work[d][c] <= kWorkCap;
        if (ok) deal = d;
    }
    const bool fits = deal >= 0;
    if (!fits) {                                        // the same decision in every CTA (same inputs)
        cluster.sync();                                 // peers are done reading this CTA's counts
        if (MODE != 0) {
            lsd_rank_all(cluster, counts, V, V, map, inv_map, keyA, valA, keyB, valB,
                         reinterpret_cast<uint32_t (*)[kDigits]>(s_dyn), &spec);
            return;
        }
        lsd_rank_all(cluster, counts, V, K, map, inv_map, keyA, valA, keyB, valB,
                     reinterpret_cast<uint32_t (*)[kDigits]>(s_dyn));
        return;
    }
    // phase 3: the keys of the inexact buckets down to the cut move into bucket order (order inside a bucket is
    // whatever the atomics make of it); ids of exact buckets down to the cut take their final rank; ids below the
    // cut are pruned here
    const int k_exact = MODE == 0 ? K : s_K;            // (MODE 1 / 2: exact ids are kept only when the cut bucket is exact)
    for (int i = w0 + lane; i < w1 + lane; i += 32 * kInFlight) {      // (every lane of the warp makes every trip)
        uint32_t c[kInFlight];
#pragma unroll
        for (int q = 0; q < kInFlight; ++q) c[q] = i + q * 32 < w1 ? __ldg(counts + i + q * 32) : 0u;
#pragma unroll
        for (int q = 0; q < kInFlight; ++q) {
            const int id = i + q * 32;
            const bool on = id < w1;
            const int b = (int)(kFine - 1 - fine_bucket(c[q]));
            const bool kept = on && b <= cut;
            const bool exact = kept && b >= first_exact;
            const unsigned group = __ballot_sync(0xffffffffu, exact);
            if (exact) {
                const unsigned peers = __match_any_sync(group, c[q]);
                const int leader = __ffs(peers) - 1;
                uint32_t before = 0;
                if (lane == leader) {
                    before = s_ws[warp][c[q]];
                    s_ws[warp][c[q]] = (uint16_t)(before + __popc(peers));
                }
                before = __shfl_sync(peers, before, leader);
                const int rk = (int)(s_next[b] + before + __popc(peers & lanemask_lt()));
                if (rk < k_exact) map[rk] = id;
                inv_map[id] = rk < k_exact ? rk : -1;
            } else if (kept) {
                pairs[atomicAdd(&s_next[b], 1u)] = ((unsigned long long)c[q] << 32) | (0xffffffffu - (uint32_t)id);
            } else if (on) {
                inv_map[id] = -1;
            }
            __syncwarp();
        }
    }
    __threadfence();
    cluster.sync();
    // phase 4: place of a key = start of its bucket + number of greater keys in the bucket.  Inside a bucket the
    // counts differ in their low bits only, so what is compared is a 32-bit word (those low bits, then ~id) held in
    // shared memory for the CTA's whole run of buckets, four to a load (neighbouring lanes mostly share a bucket:
    // the reads are broadcasts).  The 64-bit keys stay where phase 3 put them and are read from there.
    const int r0 = s_lo[deal], n = s_hi[deal] > s_lo[deal] ? s_hi[deal] - s_lo[deal] : 0;
    const unsigned long long* run = pairs + r0;
    uint32_t* s_c = reinterpret_cast<uint32_t*>(s_run);                 // [kSortCap]
    uint32_t* s_place = s_c + kSortCap;                                 // [kSortCap] MODE 1 / 2: the keys' ranks
    const int idbits = id_bits(V);
    for (int j = threadIdx.x; j < n; j += kThreads) s_c[j] = short_key(__ldcg(run + j), idbits);
    __syncthreads();
    if (MODE == 0) {
        for (int j = threadIdx.x; j < n; j += kThreads) {
            const unsigned long long key = __ldcg(run + j);
            const int b = (int)(kFine - 1 - fine_bucket((uint32_t)(key >> 32)));
            const int bs = (int)s_gstart[b] - r0, be = bs + (int)s_gsize[b];
            const int rk = r0 + bs + rank_in_bucket<false>(s_c, run, key, bs, be, idbits, nullptr);
            const int32_t v = (int32_t)(0xffffffffu - (uint32_t)key);
            if (rk < K) map[rk] = v;
            inv_map[v] = rk < K ? rk : -1;
        }
        return;
    }
    // K from the ranks.  A key of a bucket above the cut is kept whatever K turns out to be (K is at least the cut
    // bucket's first rank) and is emitted with its place; the keys of the cut bucket -- all in one CTA -- get their
    // places (and, Top-P, the token mass ranked before them), that CTA reads K off them, and then they are emitted.
    const bool owns_cut = s_cut_owner[deal] == (int)rank || (s_cut_owner[deal] < 0 && rank == 0);   // (an empty cut bucket has no owner)
    const unsigned long long mass_before = s_mass_before;
    for (int j = threadIdx.x; j < n; j += kThreads) {
        const unsigned long long key = __ldcg(run + j);
        const uint32_t cnt = (uint32_t)(key >> 32);
        const int b = (int)(kFine - 1 - fine_bucket(cnt));
        const int bs = (int)s_gstart[b] - r0, be = bs + (int)s_gsize[b];
        int r;
        if (b == cut && MODE == 1) {
            unsigned long long m = 0;
            r = rank_in_bucket<true>(s_c, run, key, bs, be, idbits, &m);
            const unsigned long long cum = mass_before + m;
            if (below(cum) && reaches(cum + cnt)) s_K = r0 + bs + r + 1;                          // exactly one key
        } else {
            r = rank_in_bucket<false>(s_c, run, key, bs, be, idbits, nullptr);
            if (b == cut && MODE == 2 && cnt >= min_count) atomicMax(&s_K, r0 + bs + r + 1);
        }
        const int rk = r0 + bs + r;
        if (b == cut) {
            s_place[j] = (uint32_t)rk;
        } else {
            const int32_t v = (int32_t)(0xffffffffu - (uint32_t)key);
            s_place[j] = 0xffffffffu;                   // emitted
            map[rk] = v;
            inv_map[v] = rk;
        }
    }
    __syncthreads();
    if (!owns_cut) return;
    const int Kf = max(1, min(V, s_K));
    if (threadIdx.x == 0) *k_out = Kf;
    for (int j = threadIdx.x; j < n; j += kThreads) {
        const uint32_t rk = s_place[j];
        if (rk == 0xffffffffu) continue;
        const int32_t v = (int32_t)(0xffffffffu - (uint32_t)__ldcg(run + j));
        if ((int)rk < Kf) map[rk] = v;
        inv_map[v] = (int)rk < Kf ? (int)rk : -1;
    }
}

}  // namespace

static cudaError_t select_smem_attr() {
    static int attr_done[64] = {0};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && attr_done[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(k_select_sort<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSelectSmem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_select_sort<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSelectSmem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_select_sort<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSelectSmem);
    if (e == cudaSuccess && dev >= 0 && dev < 64) attr_done[dev] = 1;
    return e;
}

// Top-P (mode 0) / minimum frequency (mode 1): the selection kernel in the mode that finds K on its way.
cudaError_t launch_select_cut(const uint32_t* counts, int32_t V, int mode, double pfrac, uint32_t min_count,
                              int32_t* map, int32_t* inv_map, int32_t* k_out, uint8_t* scratch, cudaStream_t s) {
    const size_t seg = align_up((size_t)V * 4, 256);
    uint32_t* keyA = reinterpret_cast<uint32_t*>(scratch);
    uint32_t* valA = reinterpret_cast<uint32_t*>(scratch + seg);
    uint32_t* keyB = reinterpret_cast<uint32_t*>(scratch + 2 * seg);
    uint32_t* valB = reinterpret_cast<uint32_t*>(scratch + 3 * seg);
    cudaError_t e = select_smem_attr();
    if (e != cudaSuccess) return e;
    if (mode == 0)
        k_select_sort<1><<<kCluster, kThreads, kSelectSmem, s>>>(counts, V, 0, map, inv_map, keyA, valA, keyB, valB, pfrac, 0u, k_out);
    else
        k_select_sort<2><<<kCluster, kThreads, kSelectSmem, s>>>(counts, V, 0, map, inv_map, keyA, valA, keyB, valB, 1.0, min_count, k_out);
    count_launch();
    return cudaGetLastError();
}

size_t select_scratch_bytes(int32_t V) { return 4 * align_up((size_t)V * 4, 256); }
size_t select_cut_scratch_bytes(int32_t V) { return select_scratch_bytes(V); }

cudaError_t launch_select_topk(const uint32_t* counts, int32_t V, int32_t K, int32_t* map,
                               int32_t* inv_map, uint8_t* scratch, cudaStream_t s) {
    const size_t seg = align_up((size_t)V * 4, 256);
    uint32_t* keyA = reinterpret_cast<uint32_t*>(scratch);
    uint32_t* valA = reinterpret_cast<uint32_t*>(scratch + seg);
    uint32_t* keyB = reinterpret_cast<uint32_t*>(scratch + 2 * seg);
    uint32_t* valB = reinterpret_cast<uint32_t*>(scratch + 3 * seg);
    cudaError_t e = select_smem_attr();
    if (e != cudaSuccess) return e;
    // (whatever K: even K = V is the selection's work when most ids were seen fewer than 1024 times -- 31 against
    // 56 us on the counts of 3 M tokens -- and costs it one bucket pass, 13 us, before the full ranking when not)
    k_select_sort<0><<<kCluster, kThreads, kSelectSmem, s>>>(counts, V, K, map, inv_map, keyA, valA, keyB, valB, 1.0, 0u, nullptr);
    count_launch();
    return cudaGetLastError();
}

}  // namespace vt
